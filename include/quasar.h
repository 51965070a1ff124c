/*
 * quasar.h — C ABI of the B200 (sm_100a) quantised verification pass.
 *
 * The library implements the verification half of one speculative-decoding
 * iteration (Quasar, arXiv 2603.01399, Section 3.1 "Verification" and
 * Section 3.3): the target decoder, holding low-bit weights, scores a block of
 * drafted tokens against its KV cache in ONE parallel forward pass, then the
 * longest draft prefix that agrees with the verifier's own top-1 choices is
 * accepted and one more token (the verifier's) is emitted.
 *
 * Weights are int8, symmetric, one fp32 step size per output channel
 * (Section 3.2, Eq. 6-8: W_int8 = Q(W, delta_w), Y ~= delta_w * (W_int8 X));
 * activations stay bf16 and accumulation is fp32.  A bf16-weight pass built
 * from the same kernels (the "BF16 verifier" the paper compares with,
 * Section 3.4 Eq. 11) is selected with weight_dtype = QUASAR_W_BF16.
 *
 * Conventions
 *  - C linkage; every function returns QUASAR_OK (0) or a negative error code
 *    and never throws or aborts.  quasar_last_error() gives a thread-local
 *    message for the last failing call of the calling thread.
 *  - Unless a parameter says "host", every pointer is DEVICE memory owned by
 *    the caller, 16-byte aligned, valid until the work queued by the call has
 *    finished.  The library allocates no device memory per call; scratch comes
 *    from a caller-provided workspace (quasar_workspace_bytes).
 *  - `stream` is a cudaStream_t passed as void*.  Unless a call says otherwise it only
 *    enqueues work (no synchronisation, no allocation); results are valid once the
 *    stream has been synchronised.  quasar_plan_create is the supported way to freeze a
 *    pass for replay: it captures the kernel-per-step form into a CUDA graph itself and
 *    keeps the persistent single-kernel form (a cooperative launch) as a plain launch.
 *  - Argument errors that the host can see are reported before anything is
 *    launched.  Errors only the device can see (a token id out of range, a
 *    malformed parent array, a sequence that would overflow its cache) set the
 *    caller's `status` word to a negative code; the offending sequence is
 *    skipped, nothing is written out of bounds and nothing traps.
 *  - Matrices are row-major with the contraction index contiguous:
 *    W is [N][K] = [d_out][d_in] (the paper's W in R^{d_out x d_in}, Section 3.2).
 */
#ifndef QUASAR_H_
#define QUASAR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define QUASAR_OK 0
#define QUASAR_ERR_INVALID_ARG (-1) /* null pointer, negative size, bad enum     */
#define QUASAR_ERR_SHAPE (-2)       /* size not supported (see each call)        */
#define QUASAR_ERR_CAPACITY (-3)    /* workspace / cache / batch limit exceeded  */
#define QUASAR_ERR_ALIGN (-4)       /* pointer not 16-byte aligned               */
#define QUASAR_ERR_CUDA (-5)        /* a CUDA runtime call failed                */
#define QUASAR_ERR_TIMEOUT (-6)     /* a bounded device-side wait ran out        */
#define QUASAR_ERR_TOKEN (-7)       /* device: token id outside [0, vocab)       */
#define QUASAR_ERR_TREE (-8)        /* device: parents[] is not a rooted forest order */

#define QUASAR_W_INT8 0
#define QUASAR_W_BF16 1

#define QUASAR_A_BF16 0 /* activations stay bf16 (weight-only quantisation)                      */
#define QUASAR_A_INT8 1 /* the paper's W8A8: every linear layer quantises its input per token    */

#define QUASAR_MAX_BLOCK 64 /* rows of one sequence's draft block (root + drafts / tree nodes) */

const char* quasar_last_error(void);

/* ------------------------------------------------------------------------
 * Offline weight preparation (Section 3.3 "Offline Weight Preparation";
 * Q(., delta) of Section 3.2 Eq. 6).  Per output channel n:
 *   delta[n] = max_k |W[n][k]| / 127   (fp32 IEEE division; 1.0f for an all-zero row)
 *   q[n][k]  = clamp(round_half_even(W[n][k] / delta[n]), -127, 127)   (fp32 division)
 * w_bf16: [N][K] bf16.  q_out: [N][K] int8.  delta_out: [N] fp32.  K % 8 == 0.
 * Bit-exact with the definition above; no fast-math anywhere on this path.
 * ---------------------------------------------------------------------- */
int quasar_quantize(const void* w_bf16, int64_t N, int64_t K, int8_t* q_out, float* delta_out, void* stream);

/* ------------------------------------------------------------------------
 * One quantised linear layer (Section 3.2 Eq. 8 / Section 3.3 Eq. 10, weight-only):
 *   Y[m][n] = delta[n] * sum_k X[m][k] * (float)W[n][k]   (+ R[m][n] if residual != NULL)
 * x: [M][K] bf16.  w: [N][K] int8 (weight_dtype = QUASAR_W_INT8) or bf16
 * (QUASAR_W_BF16, delta ignored and may be NULL).  y: [M][N], bf16 or fp32
 * (y_is_f32).  residual: [M][N] bf16 or NULL; with a residual the product is
 * first rounded to bf16, then added, then rounded again (the order the decoder
 * layer uses).  y may alias residual.  M >= 1 (rows are processed in groups of
 * at most 72), K % 16 == 0, 1 <= N <= 1048576 (QUASAR_ERR_SHAPE beyond).
 * workspace: at least quasar_linear_workspace_bytes(M, N, K) bytes; its first
 * use must find its first 64 KiB zero-filled, and every call leaves it reusable by the next call of
 * any shape (the split-K arrival counters live in those 64 KiB and reset themselves).
 * Accumulation is fp32, or better: int8 weights with more than 8 rows run on the tcgen05 tensor
 * cores (fp16 operands - exact for bf16 rows scaled by a power of two - fp32 sums in tensor
 * memory); int8 weights with at most 8 rows on a matrix of at least 128 MiB run as an exact
 * integer contraction (the activation row as 21-bit fixed point against a power of two above its
 * largest magnitude).  Which kernel runs depends only on the shape and on whether the workspace
 * has the size quasar_linear_workspace_bytes reports (a smaller one that still fits the fp32
 * kernel is accepted); the kernels agree to fp32 accumulation accuracy, not bit for bit.
 * ---------------------------------------------------------------------- */
int quasar_linear_workspace_bytes(int64_t M, int64_t N, int64_t K, size_t* bytes_out /* host */);
int quasar_linear(const void* x, const void* w, const float* delta, int32_t weight_dtype, int64_t M, int64_t N,
                  int64_t K, void* y, int32_t y_is_f32, const void* residual, void* workspace,
                  size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------
 * The paper's W8A8 form (Section 3.2 Eq. 4-8, Section 3.3 Eq. 9-10): activations are quantised
 * too, per token, after a per-channel smoothing that moves outliers from the activations into
 * the weights.  Q(., delta) is the operator of quasar_quantize throughout.
 *
 * quasar_smoothing_factors (Eq. 5, offline calibration): act_absmax fp32 [K] = max|X_j| of the
 *   layer's input over calibration data; w_bf16 [N][K].  s_out fp32 [K]:
 *     s_j = max|W_j|^(1-alpha) / max|X_j|^alpha   (fp64 arithmetic, stored as fp32; 1 where either
 *     maximum is zero).  This is the factor the activations are MULTIPLIED by in Eq. 4 / Eq. 9,
 *     i.e. the reciprocal of the expression printed as Eq. 5 (see the note in w8a8.cu).
 * quasar_quantize_weights_smoothed (Section 3.3 "Offline Weight Preparation"):
 *     W_int8 = Q(W diag(s)^-1, delta_w), W / s in fp32; s == NULL: same as quasar_quantize.
 * quasar_quantize_activations (Eq. 9, fused smoothing + quantisation): x bf16 [M][K],
 *     X_int8 = Q(X * s, delta_x), one step size per token (row), x * s in fp32; s may be NULL.
 * quasar_linear_w8a8 (Eq. 8, Eq. 10): quantises x as above into the workspace, then
 *     Y_int32 = W_int8 x X_int8 (exact), Y = Y_int32 * (delta_w[n] * delta_x[m]) in fp32
 *     (+ residual as in quasar_linear).  acc_out: int32 [M][N] or NULL - the raw accumulators,
 *     for callers that want to check them.  K % 16 == 0; workspace as for quasar_linear
 *     (first 64 KiB zero on first use), size from quasar_linear_w8a8_workspace_bytes.
 * All bit-exact in the integer codes and accumulators; K % 8 == 0 for the quantisers.
 * ---------------------------------------------------------------------- */
int quasar_smoothing_factors(const float* act_absmax, const void* w_bf16, int64_t N, int64_t K, float alpha,
                             float* s_out, void* stream);
int quasar_quantize_weights_smoothed(const void* w_bf16, const float* s, int64_t N, int64_t K, int8_t* q_out,
                                     float* delta_out, void* stream);
int quasar_quantize_activations(const void* x_bf16, const float* s, int64_t M, int64_t K, int8_t* q_out,
                                float* delta_out, void* stream);
int quasar_linear_w8a8_workspace_bytes(int64_t M, int64_t N, int64_t K, size_t* bytes_out /* host */);
int quasar_linear_w8a8(const void* x, const float* s, const int8_t* w, const float* delta_w, int64_t M, int64_t N,
                       int64_t K, void* y, int32_t y_is_f32, const void* residual, int32_t* acc_out, void* workspace,
                       size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------
 * 4-bit weights (Section 6, "Ultra-low Bit Verification", the first item of the paper's outlook;
 * the weight term of Section 3.4 drops to a quarter of the bf16 one).  The quantiser is Q of Eq. 6
 * with the range [-7, 7] and one step size per output channel and group of 128 consecutive input
 * channels; two codes per byte, the even input channel in the low nibble, two's complement.
 * quasar_quantize_int4: w_bf16 [N][K], K % 128 == 0 -> packed uint8 [N][K/2], delta fp32 [N][K/128];
 *   bit-exact with the definition (fp32 IEEE division, round-half-even, all-zero group -> delta 1).
 * quasar_linear_w4:  Y[m][n] = sum_g delta[n][g] * sum_{k in g} X[m][k] * code[n][k]  (+ residual as
 *   in quasar_linear); x bf16 [M][K]; fp32 accumulation inside a group and across groups; y bf16 or
 *   fp32; workspace from quasar_linear_w4_workspace_bytes (no zero-filling needed).
 * ---------------------------------------------------------------------- */
int quasar_quantize_int4(const void* w_bf16, int64_t N, int64_t K, uint8_t* packed_out, float* delta_out, void* stream);
int quasar_linear_w4_workspace_bytes(int64_t M, int64_t N, int64_t K, size_t* bytes_out /* host */);
int quasar_linear_w4(const void* x, const uint8_t* packed, const float* delta, int64_t M, int64_t N, int64_t K, void* y,
                     int32_t y_is_f32, const void* residual, void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------
 * quasar_linear for callers that may not allocate device memory.  (The paper has no
 * counterpart: this is a convenience of the library, not a step of the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits, for instance a plug-in
 * inside a host application that owns the whole memory pool and hands out only the input
 * and output tensors, or a latency-critical loop that must not touch the allocator (an
 * allocation can synchronise the device).  Such a caller has no workspace to pass.
 *
 * Same arithmetic, arguments and result as quasar_linear, minus the workspace: the scratch
 * of the split-K reduction lives in a fixed array of quasar_linear_static_scratch_bytes()
 * (4 MiB) inside the library, which every GPU that loads the library holds until the
 * process exits.  The call itself allocates and frees nothing.
 *  - Shapes whose scratch would exceed the array are refused with QUASAR_ERR_CAPACITY
 *    (the message gives both sizes); use quasar_linear for those.
 *  - The array is the one of the CURRENT device: on every call the current device must be the
 *    device `stream` belongs to (the library cannot check this; a mismatch hands the kernel
 *    another GPU's address).  The first call on a device looks up the array's device address;
 *    that lookup may make the runtime load the library's device code and is the only step
 *    that can allocate, so make that first call outside any stream capture.  Argument errors
 *    are reported before the lookup.
 *  - All calls on a device share the one array, and it keeps the previous call's contents
 *    (the part that must start at zero is cleared on `stream` by every call).  Two calls
 *    that may overlap on the GPU - different streams without an ordering between them -
 *    race on it; issue them on one stream or order them with events.
 * ---------------------------------------------------------------------- */
size_t quasar_linear_static_scratch_bytes(void);
int quasar_linear_static(const void* x, const void* w, const float* delta, int32_t weight_dtype, int64_t M, int64_t N,
                         int64_t K, void* y, int32_t y_is_f32, const void* residual, void* stream);

/* ------------------------------------------------------------------------
 * Model description.  The paper fixes only the linear layers; the rest of the
 * decoder layer (Section 3.3: "non-linear layers" stay in high precision) is a
 * pre-norm decoder: RMSNorm (y = x * rsqrt(mean(x^2) + eps) * g), optional
 * per-head RMSNorm of q and k over head_dim before RoPE, rotate-half RoPE
 * (pairs (i, i + head_dim/2), inv_freq_i = theta^(-2i/head_dim)), grouped-query
 * attention, SwiGLU  down(silu(gate) * up), no biases, untied LM head.
 * ---------------------------------------------------------------------- */
typedef struct quasar_config {
  int32_t n_layers;
  int32_t hidden;       /* H, multiple of 16                                  */
  int32_t n_q_heads;    /* Hq, multiple of n_kv_heads, Hq / Hkv <= 8          */
  int32_t n_kv_heads;   /* Hkv                                                */
  int32_t head_dim;     /* D: 64 or 128                                       */
  int32_t ffn;          /* F, multiple of 16                                  */
  int32_t vocab;        /* V                                                  */
  int32_t qk_norm;      /* 1: per-head RMSNorm of q and k before RoPE         */
  float rope_theta;
  float rms_eps;
  int32_t weight_dtype; /* QUASAR_W_INT8 or QUASAR_W_BF16                     */
  int32_t max_seq;      /* cache capacity S_max (positions) the RoPE table covers */
  int32_t act_dtype;    /* QUASAR_A_BF16, or QUASAR_A_INT8 (needs weight_dtype QUASAR_W_INT8; the
                           weights must then be Q(W diag(s)^-1) for the smoothing vectors below) */
  int32_t weights_in_place; /* 0: the model borrows the weight matrices and keeps a second, permuted copy for
                           the persistent single-kernel pass (twice the weight bytes).  1: the caller hands
                           the matrices over: quasar_model_create permutes each of them WHERE IT LIES into the
                           order the persistent kernel streams it (their contents are no longer row-major
                           afterwards) and keeps no copy, so the model occupies the weight bytes once - the
                           footprint Section 3.3 ("Offline Weight Preparation") promises.  Such a model
                           runs the persistent kernel only: blocks of at most 8 rows in total, no trace. */
} quasar_config;

typedef struct quasar_layer_weights {
  const void* attn_norm;  /* bf16 [H]                                             */
  const void* qkv_w;      /* [(Hq + 2 Hkv) D][H]: q heads, then k heads, then v   */
  const float* qkv_delta; /* fp32 [(Hq + 2 Hkv) D]   (NULL for bf16 weights)      */
  const void* q_norm;     /* bf16 [D] or NULL when qk_norm == 0                   */
  const void* k_norm;     /* bf16 [D] or NULL                                     */
  const void* o_w;        /* [H][Hq D]                                            */
  const float* o_delta;
  const void* mlp_norm;   /* bf16 [H]                                             */
  const void* gateup_w;   /* [2F][H]: rows [0,F) gate, rows [F,2F) up             */
  const float* gateup_delta;
  const void* down_w;     /* [H][F]                                               */
  const float* down_delta;
  /* act_dtype == QUASAR_A_INT8 only: smoothing factors of each linear layer's input (Eq. 4-5, Eq. 9),
   * fp32 over the layer's input channels, or NULL for no smoothing                                   */
  const float* qkv_smooth;    /* [H]     */
  const float* o_smooth;      /* [Hq D]  */
  const float* gateup_smooth; /* [H]     */
  const float* down_smooth;   /* [F]     */
} quasar_layer_weights;

typedef struct quasar_weights {
  const void* embed;                  /* bf16 [V][H]                               */
  const quasar_layer_weights* layers; /* HOST array of n_layers entries (device pointers inside) */
  const void* final_norm;             /* bf16 [H]                                  */
  const void* lm_w;                   /* [V][H]                                    */
  const float* lm_delta;              /* fp32 [V]                                  */
  const float* lm_smooth;             /* fp32 [H] or NULL (act_dtype == QUASAR_A_INT8 only) */
} quasar_weights;

/* KV cache of the context x_<t (Section 3.1): bf16, [L][B][Hkv][S_max][D], K
 * already rotated.  seq_len[b] = positions of sequence b that are committed. */
typedef struct quasar_kv {
  void* k;
  void* v;
  int32_t* seq_len; /* device int32 [batch]                                       */
  int32_t batch;    /* B the cache was laid out for                               */
  int32_t s_max;    /* <= config.max_seq                                          */
} quasar_kv;

typedef struct quasar_model quasar_model;

/* The model borrows every weight pointer (they must outlive it) and owns a
 * RoPE cos/sin table built in fp64 on the device.  Allocates; not capturable. */
int quasar_model_create(const quasar_config* cfg /* host */, const quasar_weights* w /* host */, quasar_model** out);
int quasar_model_destroy(quasar_model* m);

/* Bytes of scratch quasar_verify needs for batch B and T_max block rows. */
int quasar_workspace_bytes(const quasar_model* m, int32_t B, int32_t T_max, size_t* bytes_out /* host */);

/* ------------------------------------------------------------------------
 * The verification pass (Section 3.1 "Verification", Section 3.3) with greedy
 * acceptance (Eq. 2 at temperature 0: a draft token is kept while it equals the
 * verifier's top-1 prediction).
 *
 * tokens     int32 [B][T_max]; row 0 of a sequence is its last emitted token
 *            (not yet in the cache), rows 1.. are the drafted tokens (chain) or
 *            tree nodes.
 * parents    NULL for chains (row i follows row i-1); else int32 [B][T_max] with
 *            parents[b][0] = -1 and 0 <= parents[b][i] < i.  Row i sits at
 *            position seq_len[b] + depth(i) and attends to the whole cached
 *            prefix, its ancestors and itself.
 * block_len  int32 [B], 1 <= block_len[b] <= T_max <= QUASAR_MAX_BLOCK; rows
 *            beyond it are ignored (1 = one plain decode step).
 * logits_out fp32 [B][T_max][V] or NULL.  Row i predicts the token after row i.
 * accept_len int32 [B]: number of accepted DRAFT tokens, in [0, block_len-1]; -1 for a
 *            sequence that was skipped because of a device-detected error (see status).
 * bonus      int32 [B]: the verifier's token after the last accepted row (-1 if skipped).
 * accept_path int32 [B][T_max] or NULL: accept_path[b][d] = block row accepted at
 *            depth d (entry 0 is the root, entries past accept_len are -1).
 * status     int32 [1]: left untouched on success, else a negative code.
 *
 * K and V of every block row are written to cache slot seq_len[b] + row; seq_len
 * is not changed, so the call is idempotent until quasar_kv_commit.  Ties in the
 * argmax go to the lowest token id; equal sibling tokens to the lowest row.
 * ---------------------------------------------------------------------- */
int quasar_verify(quasar_model* m, const quasar_kv* kv /* host struct */, const int32_t* tokens,
                  const int32_t* parents, const int32_t* block_len, int32_t B, int32_t T_max, float* logits_out,
                  int32_t* accept_len, int32_t* bonus, int32_t* accept_path, void* workspace,
                  size_t workspace_bytes, int32_t* status, void* stream);

/* ------------------------------------------------------------------------
 * Drafting by prompt lookup (Section 4.1: the n-gram drafter of the paper's experiments; lookup
 * range K = (k_min, k_max) of Section 4.4 / Table 3).  Per sequence: for n = k_max down to k_min
 * the last n of its hist_len[b] tokens are searched for among the tokens before them; the most
 * recent earlier occurrence that is followed by at least one token wins, and the up to gamma
 * tokens after it are the draft (the longest n with such an occurrence is used).
 * history int32 [B][S] (the sequence so far, prompt included); hist_len int32 [B] (<= S);
 * draft int32 [B][gamma] (entries past draft_len are -1); draft_len int32 [B] in [0, gamma]
 * (0: nothing to look up - verify with block_len 1, a plain decode step).  1 <= k_min <= k_max.
 * ---------------------------------------------------------------------- */
int quasar_ngram_draft(const int32_t* history, const int32_t* hist_len, int32_t B, int32_t S, int32_t gamma,
                       int32_t k_min, int32_t k_max, int32_t* draft, int32_t* draft_len, void* stream);

/* ------------------------------------------------------------------------
 * Stochastic acceptance of drafted CHAINS (Section 3.1 Eq. 2-3; Section 3.3 "Lossless Rejection
 * Sampling"), applied to the logits quasar_verify wrote.  With p = softmax(logits / temperature):
 * draft i+1 (block row i+1) is accepted while r_accept[b][i] < min(1, p_i(token) / q_i(token))
 * (Eq. 2); at the first rejection next_token is drawn from norm(max(0, p_i - q_i)) (Eq. 3); if all
 * drafts are accepted it is drawn from p of the last row.  A draw is by inversion with r_sample[b]:
 * the smallest v with w_0 + ... + w_v > r_sample * sum(w).
 * logits fp32 [B][T_max][V]; tokens, block_len as in quasar_verify; q_probs fp32 [B][T_max][V] (row i:
 * the distribution draft i+1 came from) or NULL for a drafter that proposes its token with
 * certainty (q = point mass: accepted with probability p(token), residual = p without that token);
 * temperature > 0; r_accept fp32 [B][T_max] and r_sample fp32 [B], uniform in [0, 1), supplied by
 * the caller; accept_len, next_token int32 [B].  fp32 arithmetic with fixed reduction orders (bit
 * for bit repeatable); a decision that sits within rounding of its threshold may differ from an
 * fp64 evaluation.  workspace: quasar_accept_stochastic_workspace_bytes(B, T_max) bytes.
 * quasar_kv_commit takes the resulting accept_len like the greedy one.
 * ---------------------------------------------------------------------- */
int quasar_accept_stochastic_workspace_bytes(int32_t B, int32_t T_max, size_t* bytes_out /* host */);
int quasar_accept_stochastic(const float* logits, const int32_t* tokens, const int32_t* block_len, const float* q_probs,
                             int32_t B, int32_t T_max, int32_t V, float temperature, const float* r_accept,
                             const float* r_sample, int32_t* accept_len, int32_t* next_token, void* workspace,
                             size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------
 * Commit the accepted tokens (the cache reuse Section 3.1 implies between
 * iterations).  Chain (accept_path NULL): seq_len[b] += 1 + accept_len[b].
 * Tree: K,V of the accepted row at depth d move to slot seq_len[b] + d for
 * d = 1..accept_len[b], then the same bump.  The only call that changes seq_len.
 * A sequence whose accept_len is negative (skipped by quasar_verify) is left untouched:
 * its K/V rows were never written, so committing them would publish garbage.
 * ---------------------------------------------------------------------- */
int quasar_kv_commit(quasar_model* m, const quasar_kv* kv /* host struct */, const int32_t* accept_len,
                     const int32_t* accept_path, int32_t B, int32_t T_max, void* stream);

/* ------------------------------------------------------------------------
 * A verify pass frozen for replay: same arguments as quasar_verify, captured
 * once into a CUDA graph (or, when the pass is a single persistent kernel, kept
 * as that one launch), replayed with one call.  Every pointer is baked in; their
 * CONTENTS may change between launches.  quasar_plan_create captures on an
 * internal stream and synchronises it (not capturable itself).
 * ---------------------------------------------------------------------- */
typedef struct quasar_plan quasar_plan;
int quasar_plan_create(quasar_model* m, const quasar_kv* kv, const int32_t* tokens, const int32_t* parents,
                       const int32_t* block_len, int32_t B, int32_t T_max, float* logits_out, int32_t* accept_len,
                       int32_t* bonus, int32_t* accept_path, void* workspace, size_t workspace_bytes,
                       int32_t* status, quasar_plan** out);
int quasar_plan_launch(quasar_plan* p, void* stream);
int quasar_plan_destroy(quasar_plan* p);

/* The call a serving loop makes with HOST buffers: copies tokens (and parents,
 * block_len when given) from host memory into the plan's device buffers,
 * replays the plan, copies accept_len, bonus (and accept_path, status) back and
 * synchronises the stream.  Host buffers should be pinned for the copies to be
 * asynchronous.  Any host pointer except tokens_host may be NULL (that
 * transfer is skipped). */
int quasar_plan_run_host(quasar_plan* p, const int32_t* tokens_host, const int32_t* parents_host,
                         const int32_t* block_len_host, int32_t* accept_len_host, int32_t* bonus_host,
                         int32_t* accept_path_host, int32_t* status_host, void* stream);

/* ------------------------------------------------------------------------
 * Debug tap: when a trace buffer is set, quasar_verify copies every
 * intermediate tensor into it in a fixed order (see quasar_trace_bytes) so each
 * step of the pass can be compared on its own.  Pass NULL to switch it off.
 * Per call: embed [M][H]; per layer: h1 [M][H], qkv [M][(Hq+2Hkv)D] (before
 * RoPE), q [M][(Hq+2Hkv)D] (the same buffer after QK-norm + RoPE of its q part),
 * attn [M][Hq D], x_attn [M][H], act [M][F], x_mlp [M][H]; then hf [M][H].
 * All bf16, M = B * T_max rows.
 * ---------------------------------------------------------------------- */
int quasar_trace_bytes(const quasar_model* m, int32_t B, int32_t T_max, size_t* bytes_out /* host */);
int quasar_set_trace(quasar_model* m, void* trace_buf, size_t bytes);

/* Which implementation quasar_verify uses: 0 = automatic (the persistent single-kernel pass
 * when the block has at most 8 rows in total, else one kernel per step), 1 = always one kernel
 * per step, 2 = require the persistent kernel (QUASAR_ERR_SHAPE if the call does not fit it).
 * Both compute the same pass (Section 3.1, 3.3); they differ in summation order only. */
int quasar_set_path(quasar_model* m, int32_t path);

/* 1 if quasar_verify would run a block of this size as the persistent single kernel (with the
 * current quasar_set_path setting and no trace), 0 if as one kernel per step, negative on error. */
int quasar_uses_persistent_kernel(const quasar_model* m, int32_t B, int32_t T_max);

/* Every wait inside the persistent kernel (grid barrier, stage barrier, attention arrival
 * count) is bounded: after budget_ns (default 2e9) the waiting thread block sets `status` to
 * QUASAR_ERR_TIMEOUT, tells its other warps to stop waiting and returns once its own copies
 * in flight have landed; nothing traps and the context stays usable.  test_extra_arrivals is
 * for tests of that path only and must be 0 otherwise: the grid barrier then expects that many
 * arrivals more than there are thread blocks, so its first wait cannot complete and runs out. */
int quasar_set_wait_budget(quasar_model* m, uint64_t budget_ns, int32_t test_extra_arrivals);

/* Count of kernels the library has launched in this process (all calls). */
int64_t quasar_kernel_launches(void);

#ifdef __cplusplus
}
#endif
#endif /* QUASAR_H_ */
