/*
 * mrp.h -- C ABI of the B200-native MRP drafting step.
 *
 * One call of the library covers what happens between two backbone forwards of a
 * block-diffusion language model that carries a Multi-token Residual Prediction (MRP)
 * module: for every still-masked position of the active block, a chain of K lightweight
 * heads turns the backbone hidden state into a residual, the residual goes through the
 * backbone's own LM head and is added to the previous step's logits, and the new logits
 * are reduced to confidence (top-1 softmax probability), log-sum-exp and argmax; these
 * drive the reveal rules, the remask rule and draft verification.
 *
 * Conventions that hold for every entry point
 *   - All tensor pointers are DEVICE pointers owned by the caller; the library borrows
 *     them for the duration of the call (weights and workspace: for the lifetime of the
 *     context; they are not copied).  Struct pointers (configs, parameter blocks, output
 *     descriptors) are HOST pointers and are read before the call returns.
 *   - Matrices are row-major.  Weight matrices are [out_features, in_features].
 *   - Calls enqueue work on the given CUDA stream (a cudaStream_t passed as void*, NULL =
 *     the default stream) and return without synchronising.  No entry point allocates
 *     device memory; all scratch lives in the caller-provided workspace (the one exception,
 *     mrp_reveal_remask_noalloc, keeps its scratch in a fixed array inside the library).
 *   - The return value is an mrp_status.  Argument errors are detected on the host before
 *     anything is launched.  Device-side anomalies (non-finite statistics, a bounded wait
 *     that gave up, a row index outside its array, a residual outside the range the tensor-core
 *     kernels are accurate in) are OR-ed as MRP_DEV_* bits into the context's int32 device
 *     status word (mrp_fetch_status) and into the optional `status` word of the call's output
 *     descriptor; kernels never trap or spin without a limit.
 *   - Index arrays coming from the caller (row_index) are checked on the device before they
 *     are used as an address: an entry outside its range raises MRP_DEV_BAD_INDEX and the row
 *     is treated as absent (nothing is read or written through it).
 *   - A context is not thread-safe: use one context per stream.
 */
#ifndef MRP_H
#define MRP_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct mrp_ctx mrp_ctx;

typedef enum {
    MRP_OK = 0,
    MRP_ERR_INVALID_ARG = 1,   /* null pointer, size out of range, misaligned pointer   */
    MRP_ERR_UNSUPPORTED = 2,   /* shape not supported by the requested kernel family    */
    MRP_ERR_CUDA = 3,          /* a CUDA runtime / driver call failed                   */
    MRP_ERR_NOMEM = 4,         /* workspace too small, or host allocation failed        */
    MRP_ERR_NONFINITE = 5,
    MRP_ERR_TIMEOUT = 6,
    MRP_ERR_CAPACITY = 7       /* size beyond a fixed built-in capacity (mrp_reveal_remask_noalloc) */
} mrp_status;

/* Bits of the device status word. */
#define MRP_DEV_NONFINITE 1    /* a log-sum-exp came out NaN or infinite                */
#define MRP_DEV_TIMEOUT 2      /* a bounded barrier wait inside a kernel ran out        */
#define MRP_DEV_BAD_INDEX 4    /* a row_index entry was outside its array, or named a dense
                                  position twice (selection); the access was skipped      */
#define MRP_DEV_RANGE 8        /* tensor-core kernels: a residual h_k - h_0 left the range in
                                  which confidence / log-sum-exp hold their 2e-3 accuracy
                                  (see mrp_create); the results were still produced        */

typedef enum { MRP_F32 = 0, MRP_BF16 = 1 } mrp_dtype;

/* mrp_config.flags */
#define MRP_FLAG_FORCE_SIMT 1  /* bf16 context: use the CUDA-core kernels instead of the
                                  tensor-core (tcgen05) kernels; a cross-check path      */

#define MRP_FLAG_NO_PDL 2      /* launch every kernel fully serialised (no programmatic
                                  dependent launch); for timing comparisons               */
#define MRP_FLAG_ROW_MAJOR_ONLY 4   /* tensor-core family: never use the few-row kernels  */
#define MRP_FLAG_NO_CHAIN 16    /* run every step as a kernel of its own: the tensor-core family's head
                                  chain of a few-row call as one kernel per GEMM instead of one
                                  persistent kernel (likewise a layer of the token-conditioned module);
                                  the CUDA-core family's pass over a few short rows
                                  (at most 8 rows, d <= 512, (K + 1) * M <= 32) as one kernel per step
                                  instead of one cooperative kernel for the whole mrp_draft call      */
#define MRP_FLAG_REQUIRE_TENSOR_CORES 32   /* bf16 context: mrp_create fails with MRP_ERR_UNSUPPORTED
                                       instead of falling back to the CUDA-core kernels when the
                                       shape or the alignment rules out the tensor-core kernels  */
#define MRP_FLAG_TRAINING_KL 64     /* reserve workspace for mrp_draft_kl (the per-slice partial sums of
                                       the KL objective); without it that entry point returns
                                       MRP_ERR_UNSUPPORTED                                           */
#define MRP_FLAG_FP8_LM 128         /* decode-regime contexts ((n_heads + 1) * max_rows <= 32, d % 256 == 0,
                                       tensor-core shapes): the LM head runs on an 8-bit copy of W_lm made
                                       at mrp_create, e4m3 values with one power-of-two scale per
                                       vocabulary row, which halves the dominant weight stream.  The
                                       context then computes with the dequantised matrix
                                       W8[v, :] = scale[v] * e4m3(W_lm[v, :] / scale[v]),
                                       scale[v] = 2^E, E the smallest integer with max|W_lm[v, :]| <=
                                       448 * 2^E (rounding to nearest, ties to even): its results are
                                       those of mrp_draft on W8, to the usual tolerances; the difference
                                       to W_lm itself is the quantisation (relative 2^-4 per weight).
                                       Other shapes: MRP_ERR_UNSUPPORTED.  Workspace: + vocab * d bytes  */
#define MRP_FLAG_NO_CTA_PAIRS 256   /* tensor-core family: run the row-major kernels one CTA per tile instead
                                     * of two-CTA clusters that share each MMA (for comparison)             */
#define MRP_FLAG_EXACT_OPERANDS 8   /* tensor-core family: always carry the LM-head activation
                                       operand as a bf16 hi + lo pair (products exact to 2^-17),
                                       also where that doubles the tensor work for nothing.  Without
                                       it, calls with more than 32 row-steps ((K+1) * M) round that
                                       operand once to fp16 (11 significant bits) against an fp16
                                       copy of W_lm kept in the workspace: half the tensor work,
                                       confidence / log-sum-exp still within 2e-3.  The copy is
                                       exact except for |w| < 2^-17 (absolute error <= 2^-25);
                                       a W_lm with |w| > 65504 switches the mode off by itself. */

typedef struct {
    int32_t d;          /* hidden size                                                   */
    int32_t d_ff;       /* SwiGLU inner size F                                           */
    int32_t vocab;      /* vocabulary size V                                             */
    int32_t n_heads;    /* number of head weight sets handed to mrp_create               */
    int32_t max_rows;   /* largest M (masked rows per call)                              */
    int32_t max_seqs;   /* largest B (sequences, i.e. active blocks, per call)           */
    int32_t block_len;  /* largest L (positions per block)                               */
    int32_t dtype;      /* mrp_dtype of weights and hidden states; logits are fp32       */
    float rms_eps;      /* epsilon of the heads' RMSNorm                                 */
    int32_t device;     /* CUDA device ordinal the context lives on                      */
    int32_t flags;      /* MRP_FLAG_*                                                    */
} mrp_config;

/*
 * One MRP head in the reduced form this library is specified on: RMSNorm followed by a
 * SwiGLU MLP without biases,
 *     x = h * rsqrt(mean(h^2) + eps) * gamma,   r = W_down ( silu(W_gate x) * (W_up x) ).
 * r is the hidden residual (Algorithm 2: h <- h + Delta) and also the vector sent through
 * the LM head (Sec. 3.2: the module reuses the backbone's LM head to produce delta).
 * The same weight set may be listed several times (a module applied K times).
 */
typedef struct {
    const void *rms_gamma;  /* [d]        */
    const void *w_gate;     /* [d_ff, d]  */
    const void *w_up;       /* [d_ff, d]  */
    const void *w_down;     /* [d, d_ff]  */
} mrp_head_weights;

/* Bytes of device workspace a context of this configuration needs (0 on a bad config). */
size_t mrp_workspace_bytes(const mrp_config *cfg);

/*
 * Create a context.  heads: HOST array of cfg->n_heads entries holding DEVICE pointers;
 * w_lm: DEVICE [vocab, d]; workspace: DEVICE, 256-byte aligned, at least
 * mrp_workspace_bytes(cfg) bytes, owned by the caller and kept alive until mrp_destroy.
 * The bf16 tensor-core kernels need d % 64 == 0, d_ff % 64 == 0, vocab % 16 == 0 and
 * 16-byte aligned weights; other bf16 shapes run on the CUDA-core kernels (two orders of
 * magnitude slower: mrp_kernel_family tells which family a context resolved to, and
 * MRP_FLAG_REQUIRE_TENSOR_CORES turns the silent choice into MRP_ERR_UNSUPPORTED).
 * Accuracy range of the tensor-core kernels: they accumulate in the tensor cores' fp32, whose
 * error grows with the length of the contractions (d, d_ff) times the size of the sums, i.e.
 * of the residual.  Confidence and log-sum-exp stay within 2e-3 of an fp64 evaluation while
 *     d * rms(h_k - h_0) <= MRP_RANGE_LIMIT      (rms over the d entries of a row, any step k)
 * (measured: log-sum-exp off by 2.5e-4 at 11 000, 1.5e-3 at 40 000, 2.2e-3 at 98 000 for d =
 * 4096, d_ff = 8192; less at equal d * rms for shorter d_ff; the benchmark shapes sit at 8 000
 * to 16 000).  A row-step beyond the limit raises MRP_DEV_RANGE and is still computed.  The
 * CUDA-core kernels (fp32 FMA, MRP_FLAG_FORCE_SIMT) have no such limit.
 * Workspace: mrp_workspace_bytes() includes, for bf16 contexts with (n_heads + 1) * max_rows
 * > 32 and without MRP_FLAG_EXACT_OPERANDS, an fp16 copy of W_lm (2 * vocab * d bytes, made
 * here with one blocking pass over W_lm): the price of the one-pass LM head above 32 row-steps.
 * On success *out receives the context.  Errors: INVALID_ARG, UNSUPPORTED, NOMEM, CUDA.
 */
#define MRP_RANGE_LIMIT 32768.0f
int mrp_create(const mrp_config *cfg, const mrp_head_weights *heads, const void *w_lm,
               void *workspace, size_t workspace_bytes, mrp_ctx **out);

/* Release the host-side context (the workspace stays the caller's).  NULL is allowed. */
void mrp_destroy(mrp_ctx *ctx);

/*
 * Outputs of mrp_draft.  conf/lse/token (and margin) are step-major [(K+1), M]: entry
 * k*M + m is masked row m after k MRP steps; k = 0 is the backbone's own logits.
 *   conf   = top-1 softmax probability (Sec. 2: the "confidence" of a position)
 *   lse    = log-sum-exp of the logit row
 *   token  = argmax, lowest token id on exact ties
 *   margin = top-1 minus top-2 logit (optional, NULL = skip)
 *   logits_out = optional [K, M, V] fp32: l_k for k = 1..K; NULL = the V-wide rows are
 *                never written to memory
 *   hidden_out = optional [M, d] fp32: h after step K; NULL = skip
 *   status = optional device int32 that receives MRP_DEV_* bits (OR-ed, never cleared)
 *   conf_first = optional [(K+1), M]: softmax probability, under step k's logits, of the token
 *            that is on top at step 0 (the token a reveal at step 0 commits); equals conf where
 *            the argmax has not moved; read by remask_policy 2 of mrp_reveal_remask; NULL = skip
 */
typedef struct {
    float *conf;
    float *lse;
    int32_t *token;
    float *margin;
    float *logits_out;
    float *hidden_out;
    int32_t *status;
    float *conf_first;
} mrp_draft_out;

/*
 * The drafting pass (Algorithm 2, lines "for k = 1..K": Delta,delta <- g(h); h <- h+Delta;
 * l <- l+delta; likewise Algorithm 3 "MRP drafting" and Algorithm 4 "MRP forward").
 *   hidden  [n_rows, d]   backbone hidden states, dtype of the context
 *   logits0 [n_rows, V]   backbone logits, fp32
 *   row_index [M] int32   rows of hidden/logits0 that are masked positions (dense position
 *                         b*L+i of each masked row), or NULL for rows 0..M-1.  Every entry
 *                         must lie in [0, n_rows), n_rows as set by mrp_set_input_rows; an entry
 *                         outside raises MRP_DEV_BAD_INDEX, nothing is read through it and the
 *                         row's statistics are those of an all-zero hidden state and logit row
 *   M in [0, max_rows], K in [0, n_heads] (head k uses weight set k-1)
 * Step k's logits are l_0 + W_lm (h_k - h_0), which equals the per-step accumulation
 * l <- l + W_lm Delta by linearity of the LM head.  Errors: INVALID_ARG, CUDA.
 */
int mrp_draft(mrp_ctx *ctx, const void *hidden, const float *logits0, const int32_t *row_index,
              int32_t M, int32_t K, const mrp_draft_out *out, void *cuda_stream);

/*
 * mrp_draft with the backbone logits stored as bf16: logits0 [n_rows, V] bf16 (16-byte aligned),
 * half the bytes of the largest input (Algorithm 2, "h, l <- f(x_t)": engines that keep their LM-head
 * output in the model's 16-bit type).  The values are taken exactly as stored (promoted to fp32);
 * everything else, outputs and tolerances included, as mrp_draft.  Errors: INVALID_ARG, CUDA.
 */
int mrp_draft_bf16_logits(mrp_ctx *ctx, const void *hidden, const void *logits0_bf16,
                          const int32_t *row_index, int32_t M, int32_t K, const mrp_draft_out *out,
                          void *cuda_stream);

/*
 * The drafting pass when the backbone hands over hidden states only.  In Algorithm 2 the
 * hidden states and the logits come out of the same forward ("h, l <- f(x_t)") and the module
 * reuses the backbone's LM head (Sec. 3.2); here that head is applied once for both: the pass
 * over W_lm that produces the residual logits also produces the base logits
 *     l_0 = W_lm n_0,   n_0 = h_0                               (final_norm_gamma == NULL)
 *                       n_0 = RMSNorm(h_0; rms_eps) * final_norm_gamma   (hidden states taken
 *                                                  before the backbone's final norm)
 * and step k's logits are W_lm (n_0 + h_k - h_0).  No [n_rows, V] input is read, and the backbone
 * needs no LM-head pass of its own for these rows.
 *   final_norm_gamma [d] in the context's dtype, or NULL; the other arguments and the outputs
 *   are those of mrp_draft.  Errors: INVALID_ARG, CUDA.
 */
int mrp_draft_from_hidden(mrp_ctx *ctx, const void *hidden, const void *final_norm_gamma,
                          const int32_t *row_index, int32_t M, int32_t K, const mrp_draft_out *out,
                          void *cuda_stream);

/*
 * The drafting pass with the training objective fused into the LM-head epilogue (Algorithm 1, last
 * lines; Eq. (3); Sec. 4.1: K unrolled iterations, uniform per-step weight, forward direction,
 * temperature 1, masked positions only).  Besides everything mrp_draft computes,
 *     kl[(k-1)*M + m] = KL( softmax(teacher[k-1, m, :]) || softmax(l_k[m, :]) ),   k = 1..K,
 * where l_k = l_0 + W_lm (h_k - h_0) are the corrected logits of unrolled step k and teacher holds the
 * frozen backbone's logits on the sequence with that step's ground-truth tokens revealed (l_{t-1} in
 * the paper's one-step notation).  The two log-sum-exps and the cross term
 * sum_v softmax(teacher)_v (teacher_v - l_v) are accumulated online, tile by tile, next to the
 * softmax statistics: neither V-wide row is ever written.
 *   teacher [K, M, V] fp32 DEVICE, rows compacted like the outputs (row (k-1)*M + m)
 *   kl      [K, M]    fp32 DEVICE
 * The other arguments are those of mrp_draft.  The LM head runs on exact (bf16 hi + lo) operands
 * whatever the context's flags.  Needs a context created with MRP_FLAG_TRAINING_KL and K >= 1.
 * Errors: INVALID_ARG, UNSUPPORTED, CUDA.  (The backward pass is outside this library.)
 */
int mrp_draft_kl(mrp_ctx *ctx, const void *hidden, const float *logits0, const float *teacher,
                 const int32_t *row_index, int32_t M, int32_t K, const mrp_draft_out *out, float *kl,
                 void *cuda_stream);

/*
 * The token-conditioned MRP module (Sec. 3.2; Fig. 1(a,c); Algorithm 2, "Delta, delta <- g(x_t, h)"),
 * one application per call so that the caller can reveal tokens between MRP steps: unlike the reduced
 * head above, this module reads the embeddings of the tokens revealed so far, so step k + 1 depends on
 * the reveals of step k and the LM head runs once per step.
 * The paper fixes the parts and leaves the details open; the form implemented (one MRP step per call:
 * the module itself as one cooperative tensor-core kernel per step for up to 64 positions on tensor-core
 * contexts (d % 128 == 0, at most 4 layers, 16-byte aligned matrices), one tensor-core kernel per matrix product
 * above that; on other contexts one cooperative CUDA-core kernel per step when B * L <= 4, else one CUDA-core kernel
 * per product; the context's own LM-head kernels behind it):
 *     e_i = emb[x_i]  (emb[mask_token] where x_i = -1);   z_i = W_proj [h_i ; e_i]
 *     n_layers times:  z += W_o Attn(RMSNorm(z) g_attn),  attention over the positions of the same block,
 *                      bidirectional, n_attn_heads heads, no positional term;
 *                      z += W_down( silu(W_gate n) * (W_up n) ),  n = RMSNorm(z) g_mlp
 *     Delta_i = z_i;   h_i <- h_i + Delta_i  (every position);   l_i <- l_i + W_lm Delta_i  (masked rows)
 * All matrices row-major [out, in] in the context's dtype, no biases.
 */
typedef struct {
    const void *g_attn, *w_q, *w_k, *w_v, *w_o;     /* [d], [d, d] x 4        */
    const void *g_mlp, *w_gate, *w_up, *w_down;     /* [d], [d_ff, d] x 2, [d, d_ff] */
} mrp_module_layer;

typedef struct {
    int32_t n_layers;               /* D (the paper: 3); 0 = the fusion projection alone          */
    int32_t n_attn_heads;           /* divides d                                                   */
    int32_t mask_token;             /* row of emb that stands for a masked position                */
    int32_t emb_rows;               /* rows of emb: tokens are checked against it on the device     */
    const void *emb;                /* [emb_rows, d] frozen token embeddings                        */
    const void *w_proj;             /* [d, 2 d]                                                     */
    const mrp_module_layer *layers; /* HOST array [n_layers] of DEVICE pointers                     */
} mrp_module_weights;

/* Bytes of additional device workspace the module needs on this context (0 on bad arguments). */
size_t mrp_module_workspace_bytes(const mrp_config *cfg, const mrp_module_weights *w);

/*
 * Attach a module to a context (weights and workspace borrowed until mrp_destroy or the next attach;
 * workspace DEVICE, 256-byte aligned, at least mrp_module_workspace_bytes).  Errors: INVALID_ARG, NOMEM.
 */
int mrp_module_attach(mrp_ctx *ctx, const mrp_module_weights *w, void *workspace, size_t workspace_bytes);

/*
 * One MRP step of the attached module over B blocks of L positions.
 *   tokens   [B*L] int32   the sequence x_t of the active blocks: token id, or -1 where still masked; an id
 *                          outside [0, emb_rows) raises MRP_DEV_BAD_INDEX and is read as masked
 *   hidden0  [B*L, d]      backbone hidden states h_0 (context dtype)
 *   h_state  [B*L, d] fp32 running hidden states h, in/out: h <- h + Delta; with first_step != 0 the call
 *                          first sets it to h_0, so the caller never converts
 *   logits0, row_index, M  as mrp_draft (row_index entries in [0, B*L))
 *   out      conf / lse / token (margin, conf_first optional) are [2, M]: entry 0 the backbone's own
 *            logits, entry 1 the logits after this step, l_0 + W_lm (h - h_0), which by linearity is the
 *            running sum l <- l + delta of Algorithm 2; hidden_out optional [M, d]; logits_out [1, M, V]
 * The caller reveals from entry 1 (mrp_reveal_remask with K = 0 on it, mrp_commit), updates tokens and
 * calls again.  On a context created with MRP_FLAG_FP8_LM the step's LM-head pass runs on the 8-bit copy of
 * W_lm, like mrp_draft's (the module's own matrices stay in the context dtype): with one LM-head pass per MRP
 * step instead of one per backbone forward, that stream weighs K times as much here.
 * Errors: INVALID_ARG, UNSUPPORTED (no module attached), CUDA.
 */
int mrp_module_step(mrp_ctx *ctx, const int32_t *tokens, const void *hidden0, float *h_state,
                    const float *logits0, const int32_t *row_index, int32_t M, int32_t B, int32_t L,
                    int32_t first_step, const mrp_draft_out *out, void *cuda_stream);

/*
 * mrp_module_step with the training objective of that step fused into its LM-head pass (Algorithm 1: the
 * module g is what the objective trains; Eq. (3); Sec. 4.1):
 *     kl[m] = KL( softmax(teacher[m, :]) || softmax(l[m, :]) ),   l = l_0 + W_lm (h - h_0) after this step,
 * teacher the frozen backbone's logits on the sequence with this step's ground-truth tokens revealed, accumulated
 * online next to the softmax statistics as in mrp_draft_kl.
 *   teacher [M, V] fp32 DEVICE, rows compacted like the outputs;   kl [M] fp32 DEVICE
 * The other arguments are those of mrp_module_step.  Needs a context created with MRP_FLAG_TRAINING_KL (and
 * without MRP_FLAG_FP8_LM).  Errors: INVALID_ARG, UNSUPPORTED, CUDA.  (The backward pass is outside this library.)
 */
int mrp_module_step_kl(mrp_ctx *ctx, const int32_t *tokens, const void *hidden0, float *h_state,
                       const float *logits0, const float *teacher, const int32_t *row_index, int32_t M, int32_t B,
                       int32_t L, int32_t first_step, const mrp_draft_out *out, float *kl, void *cuda_stream);

/*
 * The clean prefix of the module's attention (Fig. 1(c): a new block is decoded given the committed clean
 * prefix, under the attention pattern of training, where a block attends to itself and to the clean blocks in
 * front of it).  What a block sees of its prefix are the keys and values the module's own layers produced for
 * the prefix positions; the caller keeps them, per module layer, in a cache
 *     k, v   DEVICE [max_seqs, n_attn_heads, prefix_cap, d / n_attn_heads], context dtype, 16-byte aligned
 *            (head-major: the rows an attention head reads are one contiguous run)
 * of which sequence b (the b-th block of an mrp_module_step call) uses the first prefix_len[b] rows per head:
 * position i of block b then attends to those rows and to the L positions of its block in one softmax.
 *   layers      HOST array [n_layers] of the caches' DEVICE pointers (copied); NULL detaches the prefix
 *   prefix_len  DEVICE [max_seqs] int32, read by every following mrp_module_step (the caller may change the
 *               values between calls); an entry outside [0, prefix_cap] raises MRP_DEV_BAD_INDEX and is
 *               clamped
 *   append      != 0: every following mrp_module_step also stores the keys and values of its own L positions,
 *               rounded to the context dtype, in rows prefix_len[b] .. prefix_len[b] + L - 1 of sequence b's
 *               slabs (what the caller does once a block is committed, with all its tokens revealed, before it
 *               raises prefix_len[b] by L); a block that does not fit raises MRP_DEV_BAD_INDEX and stores
 *               nothing.  The rows stored by a call are not among the rows it reads.
 * Needs d / n_attn_heads <= 256.  With a prefix attached the module step runs as one cooperative tensor-core
 * kernel where it does without (up to 64 positions), else as one kernel per matrix product.
 * Errors: INVALID_ARG, UNSUPPORTED (no module attached, or heads wider than 256), NOMEM.
 */
typedef struct {
    void *k, *v;
} mrp_module_kv;

int mrp_module_set_prefix(mrp_ctx *ctx, const mrp_module_kv *layers, const int32_t *prefix_len, int32_t prefix_cap,
                          int32_t append);

typedef enum { MRP_SELECT_STATIC = 0, MRP_SELECT_DYNAMIC_REMASK = 1 } mrp_select_mode;

typedef struct {
    int32_t mode;             /* mrp_select_mode                                         */
    float tau;                /* confidence threshold (dynamic mode)                     */
    int32_t r_reveal;         /* static: positions revealed from the backbone step k=0   */
    int32_t r_draft;          /* static: positions drafted per MRP step k>=1             */
    int32_t use_cap;          /* dynamic: cap |R| at min(max(floor(0.7 n),5),L), Sec.4.4
                                 (the setting of the paper's dynamic-mode experiments)   */
    int32_t remask_policy;    /* which updated quantity revokes a member of R (Algorithm 4
                                 remask step; the paper has K = 1 and the top-1 probability):
                                 0 = min over steps 1..K of the updated confidence < tau,
                                 1 = updated confidence of step K < tau,
                                 2 = min over steps 1..K of conf_first (probability of the
                                     token revealed at step 0) < tau,
                                 3 = the argmax differs from the revealed token at some
                                     step 1..K                                            */
    int32_t ensure_progress;  /* keep at least one reveal per block                      */
    const float *conf_first;  /* DEVICE [(K+1), M], mrp_draft_out.conf_first: read by
                                 remask_policy 2 only, NULL otherwise                     */
} mrp_select_params;

/*
 * Outputs of mrp_reveal_remask; every element is written on every call.
 *   reveal_mask [B*L] int8  static: positions picked at step 0; dynamic: the reveal set R
 *   remask_mask [B*L] int8  dynamic: members of R revoked by the MRP-updated confidence
 *   out_token   [B*L] int32 token committed or drafted at the position, -1 otherwise
 *   step_of     [B*L] int8  step k at which the position was taken, -1 otherwise
 *   draft_pos, draft_tok [B, Kd] int32, Kd = K * r_draft: block positions and tokens of the
 *               drafts (steps k >= 1) in draft order, -1 padded
 *   draft_len   [B] int32
 *   status      optional device int32: MRP_DEV_BAD_INDEX is OR-ed in when a row_index entry
 *               is outside [0, B*L) (the row is ignored) or names a position a second time (the
 *               row listed last keeps the position)
 */
typedef struct {
    int8_t *reveal_mask;
    int8_t *remask_mask;
    int32_t *out_token;
    int8_t *step_of;
    int32_t *draft_pos;
    int32_t *draft_tok;
    int32_t *draft_len;
    int32_t *status;          /* optional device int32 receiving MRP_DEV_* bits, NULL = none */
} mrp_select_out;

/*
 * Reveal selection and remasking from the per-step statistics of mrp_draft.
 *   STATIC (Algorithm 2, the reveal step at k = 0..K; Algorithm 3, the draft step after each
 *   MRP update; Sec. 4.1 static denoising): for k = 0..K take the r
 *   most confident still-masked positions of each block under step k (confidence
 *   descending, position ascending on ties); k = 0 picks are reveals, k >= 1 are drafts.
 *   DYNAMIC_REMASK (Algorithm 4; Sec. 4.1 dynamic denoising; Sec. 4.4 cap): R = masked
 *   positions with conf_0 >= tau (the most confident one if none and ensure_progress;
 *   the cap's most confident ones if use_cap and |R| exceeds it); remask members of R whose
 *   updated confidence (remask_policy; variants 2 and 3 follow the revealed token instead of
 *   the top one) is < tau; if that revokes all of R and ensure_progress, the most confident
 *   member stays.  Comparisons are fp32.
 * conf, token: [(K+1), M]; row_index [M] (unique, < B*L) or NULL; 1 <= L <= block_len,
 * 1 <= B <= max_seqs.  Errors: INVALID_ARG, CUDA.
 */
int mrp_reveal_remask(mrp_ctx *ctx, const float *conf, const int32_t *token,
                      const int32_t *row_index, int32_t M, int32_t K, int32_t B, int32_t L,
                      const mrp_select_params *params, const mrp_select_out *out,
                      void *cuda_stream);

/*
 * Draft verification (Algorithm 3: a drafted position is rejected where the backbone's
 * argmax differs from the draft; Figure 1(d): candidate k embeds the first k drafts, so a
 * draft only counts while all earlier drafts were accepted).
 *   draft_tok, verify_tok [B, Kd] int32; draft_len [B] int32 (slots >= draft_len ignored)
 *   positionwise = 0: accept_len[b] = number of leading matches, accept_mask cleared from the
 *                     first mismatch on;  1: per-slot matches and their count
 *   accept_len [B] int32, accept_mask [B, Kd] int8.  Errors: INVALID_ARG, CUDA.
 */
int mrp_verify(mrp_ctx *ctx, const int32_t *draft_tok, const int32_t *verify_tok,
               const int32_t *draft_len, int32_t B, int32_t Kd, int32_t positionwise,
               int32_t *accept_len, int8_t *accept_mask, void *cuda_stream);

/*
 * Block state kept on the device between backbone forwards, and its transition x_t -> x_{t-1}.
 *   tokens       [B*L] int32, in/out: token committed at the position, -1 while it is masked
 *   row_index    [B*L] int32, out: dense positions b*L+i still masked after the call, ascending
 *                (its first *n_masked entries; the argument of the next mrp_draft and
 *                mrp_reveal_remask)
 *   n_masked     [1] int32, out
 *   block_masked [B] int32, out: positions still masked per block (0 = the block is done)
 */
typedef struct {
    int32_t *tokens;
    int32_t *row_index;
    int32_t *n_masked;
    int32_t *block_masked;
} mrp_block_state;

/*
 * Apply the outcome of one pass to the block state (the closing lines of Algorithms 2-4).
 *   accept_mask == NULL: every position the selection took (sel->out_token >= 0) is unmasked
 *     with that token: the reveals of all steps in direct decoding (Algorithm 2, reveal step
 *     at k = 0..K), and in the dynamic regime the members of R that survived remasking
 *     (Algorithm 4, remask step).
 *   accept_mask [B, Kd] int8 (from mrp_verify; speculative decoding, Algorithm 3): the step-0
 *     reveals are unmasked; drafted position sel->draft_pos[b, s] takes sel->draft_tok[b, s]
 *     only where accept_mask[b, s] != 0 (Algorithm 3, rejection step: a rejected draft stays
 *     masked).
 * Positions that already hold a token are never changed.  sel is the mrp_select_out of this
 * pass (reveal_mask and remask_mask are not read); Kd as in mrp_reveal_remask; 1 <= B <=
 * max_seqs, 1 <= L <= block_len.  Errors: INVALID_ARG, CUDA.
 */
int mrp_commit(mrp_ctx *ctx, const mrp_select_out *sel, const int8_t *accept_mask, int32_t B,
               int32_t L, int32_t Kd, const mrp_block_state *state, void *cuda_stream);

/*
 * mrp_reveal_remask without a context and without any allocation (the paper has no
 * counterpart: this is a packaging variant of the call above, same rules, same outputs).
 *
 * For callers that cannot allocate device memory and therefore cannot hand mrp_create a
 * workspace: an engine whose own pool already owns the whole GPU, a plugin running inside a
 * foreign CUDA context, a latency path on which cudaMalloc (which may synchronise the device)
 * is off limits.  The one piece of scratch the selection needs, the map from dense block
 * position to masked row, lives in a fixed array inside the library instead: 4 bytes x
 * MRP_NOALLOC_MAX_POSITIONS = 256 KiB of device memory on every GPU that loads the library,
 * held until the process exits.
 *   - B * L must not exceed MRP_NOALLOC_MAX_POSITIONS, else MRP_ERR_CAPACITY (nothing is
 *     launched); L <= 1024.  All other arguments, layouts and errors as mrp_reveal_remask;
 *     the caller still owns every input and output buffer.
 *   - Works on the CURRENT device and CUDA context, which must be those of cuda_stream and of
 *     the buffers.
 *   - The first call in each (device, CUDA context) looks up the array's device address
 *     (cudaGetSymbolAddress; the address of a module variable belongs to a context, so a second
 *     context on the same device gets its own look-up); make that first call outside of any
 *     stream capture.  Later calls only enqueue a memset and two kernels.  Never calls
 *     cudaMalloc / cudaFree.
 *   - row_index entries outside [0, B*L) are skipped and duplicates resolved exactly as in
 *     mrp_reveal_remask (MRP_DEV_BAD_INDEX in out->status if given): nothing is written
 *     outside the part of the array the call uses.
 *   - All calls on a device share the one array.  Each call re-initialises the part it uses,
 *     so earlier calls leave nothing behind, but two calls that may overlap on the GPU
 *     (different streams, no ordering between them) race on it: serialise them.
 */
#define MRP_NOALLOC_MAX_POSITIONS 65536
int mrp_reveal_remask_noalloc(const float *conf, const int32_t *token, const int32_t *row_index,
                              int32_t M, int32_t K, int32_t B, int32_t L,
                              const mrp_select_params *params, const mrp_select_out *out,
                              void *cuda_stream);

/*
 * Self-test of the bounded waits (no counterpart in the paper).  Every wait inside the kernels
 * (on an mbarrier, on another CTA) gives up after a fixed number of cycles, raises
 * MRP_DEV_TIMEOUT in the status word and lets the kernel return, so that a lost signal can never
 * hang the GPU.  This call launches one thread that waits, with the same helper and the same
 * limit (about 1.5 s) as the real kernels, for a barrier nobody completes.  After
 * synchronising, *status (DEVICE int32, may be NULL) and the context's own status word carry
 * MRP_DEV_TIMEOUT; the context stays usable.  Errors: INVALID_ARG, CUDA.
 */
int mrp_selftest_wait_timeout(mrp_ctx *ctx, int32_t *status, void *cuda_stream);

/*
 * Number of rows of the `hidden` / `logits0` arrays handed to the following mrp_draft and
 * mrp_draft_from_hidden calls: the range row_index entries are checked against on the device
 * (no counterpart in the paper).  Default, and largest value: max(max_rows, max_seqs *
 * block_len).  Errors: INVALID_ARG.
 */
int mrp_set_input_rows(mrp_ctx *ctx, int32_t n_rows);

/*
 * Copy the context's device status word (MRP_DEV_* bits OR-ed by every call on the context
 * since creation or the last clearing fetch) to dst, a DEVICE int32, as an operation on
 * cuda_stream ordered behind the calls already enqueued there; clear != 0 then resets the word.
 * Never synchronises.  Errors: INVALID_ARG, CUDA.
 */
int mrp_fetch_status(mrp_ctx *ctx, int32_t *dst, int32_t clear, void *cuda_stream);

/*
 * The 8-bit copy of the LM head of a context created with MRP_FLAG_FP8_LM: *codes receives the DEVICE
 * pointer to the e4m3 bytes [vocab, d], *scales the DEVICE pointer to the fp32 row scales [vocab]
 * (both inside the workspace, valid for the context's life).  Errors: INVALID_ARG, UNSUPPORTED.
 */
int mrp_quantised_lm_head(mrp_ctx *ctx, const uint8_t **codes, const float **scales);

/*
 * Let mrp_draft wait for the base logits separately from the hidden states.  In Algorithm 2
 * ("h, l <- f(x_t)") the logits are the last thing the backbone forward produces, and the head
 * chain needs only h: an engine can run its own LM head (or, with host buffers, the copy of
 * logits0) on another stream while the head chain runs.  After this call every mrp_draft on
 * the context enqueues a wait for cuda_event (a cudaEvent_t the caller records, before calling
 * mrp_draft, on the stream that produces logits0) immediately before the LM-head kernel, and
 * reads logits0 nowhere earlier.  NULL restores the default (logits0 ready when mrp_draft is
 * called).  mrp_draft_from_hidden ignores the event.  Errors: INVALID_ARG.
 */
int mrp_set_logits0_event(mrp_ctx *ctx, void *cuda_event);

/* Number of kernels the last mrp_draft / mrp_reveal_remask / mrp_verify call on this
 * context launched (for accounting in benchmarks). */
int32_t mrp_last_launch_count(const mrp_ctx *ctx);

/*
 * Per-phase timing of mrp_draft for benchmarks (no counterpart in the paper).  While enabled,
 * every mrp_draft call records CUDA events on its stream around three phases: 0 = row gather
 * and head chain, 1 = fused LM-head kernel, 2 = combine.  mrp_profile_read must be called
 * after the stream has been synchronised; it returns the summed milliseconds of each phase
 * over the calls since the last read (the most recent 1024 at most) in ms_phase[3] (HOST),
 * their number in *n_calls (HOST), and restarts the count.  Enabling creates CUDA events
 * (no device memory); disabling destroys them.  Errors: INVALID_ARG, NOMEM, CUDA.
 */
int mrp_profile_enable(mrp_ctx *ctx, int32_t enable);
int mrp_profile_read(mrp_ctx *ctx, float *ms_phase, int32_t *n_calls);

/* Detail of the last failed call on this context (which CUDA call, its error string); an
 * empty string if the last mrp_draft succeeded.  The pointer stays valid until mrp_destroy. */
const char *mrp_last_error(const mrp_ctx *ctx);

/* Name of the kernel family a bf16/fp32 context resolved to: "simt" or "tcgen05". */
const char *mrp_kernel_family(const mrp_ctx *ctx);

const char *mrp_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* MRP_H */
