// Internal declarations shared by the translation units of libmrp_b200.so.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include "mrp.h"

namespace mrp {

// Partial softmax statistics of one (step, row) over a slice of the vocabulary.
struct __align__(16) Partial {
    float mx;      // largest logit of the slice
    float sum;     // sum of exp(logit - mx) over the slice
    int32_t idx;   // lowest token id attaining mx
    float second;  // second largest logit of the slice (-inf if none)
};

// Partial sums of the KL objective of one (step, row) over a slice of the vocabulary: with t the
// teacher logits and l the corrected logits, mx = max_v t_v, sum = sum_v exp(t_v - mx),
// cross = sum_v exp(t_v - mx) (t_v - l_v).  KL = cross / sum - (mx + ln sum) + lse(l).
struct __align__(16) KlPartial {
    float mx, sum, cross, pad;
};

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Regions of the caller-provided workspace (byte offsets, each 256-byte aligned).
struct WorkspaceLayout {
    size_t status;      // int32[64]: device status word (first element)
    size_t h0f;         // fp32 [max_rows, d]       gathered h_0
    size_t hcur;        // fp32 [max_rows, d]       residual stream h_k
    size_t xg;          // [max_rows, d]            head input operand (fp32 simt / bf16 tc)
    size_t act;         // [max_rows, F]            SwiGLU activations (fp32 simt / bf16 tc)
    size_t xt;          // [(n_heads+1)*max_rows, d] stacked LM-head operand rows h_k - h_0
    size_t sumsq;       // fp32 [kSumsqSlices, max_rows] per-CTA partial sums of squares
    size_t partials;    // Partial [n_slices_max, (n_heads+1)*max_rows]
    size_t dense_row;   // int32 [max_seqs*block_len] dense position -> masked row or -1
    size_t sk_scratch;  // fp32 [CTAs][r_pad][128] partial accumulators of the few-row head kernels
    size_t sk_counters; // int32 [kSkMaxTiles] arrivals per weight tile (zero between launches)
    size_t ssq_fix;     // uint64 [5][128]: sums of squares per (head, row) in 2^-24 fixed point (chain kernel)
    size_t w16;         // fp16 [V, d] copy of the LM head (0 bytes unless the fp16 LM path can run)
    size_t xt16;        // fp16 [n_heads*max_rows, d] rows h_k - h_0 for that path
    size_t kl_partials; // KlPartial [n_slices_max, n_heads*max_rows] (0 bytes without MRP_FLAG_TRAINING_KL)
    size_t w8;          // e4m3 [V, d] copy of the LM head, w8_scale fp32 [V]; xq e4m3 [4 limbs * 32 rows, d] operand
    size_t w8_scale;    //   limbs, x8_scale fp32 [32] (all 0 bytes without MRP_FLAG_FP8_LM)
    size_t xq;
    size_t x8_scale;
    bool has_f16;
    size_t total;
    int32_t n_slices_max;
};

constexpr int kSumsqSlices = 512;
constexpr int kSkMaxTiles = 4096;     // weight tiles of a few-row head kernel
constexpr int kSkScratchBytes = 192 * 128 * 128 * 4;   // partial accumulators of split few-row head kernels
constexpr int kSimtSliceV = 128;      // vocabulary entries per SIMT LM-head slice
constexpr int kSimtMaxBlocks = 592;   // SIMT LM-head grid cap (4 per SM)
constexpr int kF16MinRowSteps = 33;   // fp16 LM-head operands from this many row-steps (K+1)*M on,
                                      // i.e. wherever the row-major LM-head kernel runs

WorkspaceLayout workspace_layout(const mrp_config &cfg);

struct Ctx {
    mrp_config cfg;
    mrp_head_weights *heads;   // host array [n_heads] of device pointers
    const void *w_lm;
    char *ws;
    WorkspaceLayout lay;
    bool use_tc;
    bool use_f16_lm;           // the fp16 copy of W_lm exists and is usable
    bool use_fp8_lm;           // MRP_FLAG_FP8_LM: the LM head is the e4m3 copy in the workspace
    // Set per call by mrp_draft_from_hidden: no base logits are given (logits0 == nullptr); the
    // LM-head pass computes them as W_lm n_0, n_0 = h_0 or RMSNorm(h_0) * final_gamma.
    bool from_hidden;
    const void *final_gamma;
    cudaEvent_t l0_event;      // mrp_set_logits0_event: awaited right before the LM-head kernel, or nullptr
    int input_rows;            // rows of the caller's hidden / logits0 arrays: row_index entries must be below
    bool l0_bf16;              // set per call by mrp_draft_bf16_logits: logits0 points to bf16 values
    const float *teacher;      // set per call by mrp_draft_kl: teacher logits [K, M, V], else nullptr
    float *kl_out;             // [K, M]
    // Row offset of the bf16 lo block behind the hi block in this call's operand buffers: M and
    // (K+1)M for the row-major kernels, the padded row count for the few-row kernels (which then
    // fetch hi and lo rows of a k-chunk with one TMA box).
    int lo_x, lo_xt;
    int32_t launches;
    int sm_count;
    void *tc_state;            // tensor-core path state (tensor maps), owned by tc_*.cu
    // Optional per-phase timing of mrp_draft (CUDA events on the call's stream).
    // the token-conditioned module attached with mrp_module_attach (weights and workspace borrowed)
    bool has_module;
    mrp_module_weights module;
    mrp_module_layer *module_layers;   // host copy [n_layers]
    char *module_ws;
    // the clean prefix of the module's attention (mrp_module_set_prefix): per layer the device pointers of the
    // key / value cache [max_seqs][n_attn_heads][prefix_cap][d / n_attn_heads] (context dtype), host copy; lengths per
    // sequence on the device
    bool has_prefix;
    mrp_module_kv *prefix_layers;
    const int32_t *prefix_len;
    int prefix_cap;
    bool prefix_append;
    char err[192];             // detail of the last failure ("" if none)
    bool prof_enabled;
    cudaEvent_t *prof_events;  // [kProfSlots][kProfMarks]
    int64_t prof_calls;
};

// Records where a CUDA call failed; returns the error unchanged.
inline cudaError_t note_err(Ctx *c, cudaError_t e, const char *where)
{
    if (e != cudaSuccess) snprintf(c->err, sizeof(c->err), "%s: %s", where, cudaGetErrorString(e));
    return e;
}

constexpr int kProfSlots = 1024;
constexpr int kProfMarks = 4;   // start, after head chain, after LM head, after combine

// The base logits may become ready later than the hidden states (mrp_set_logits0_event).
inline cudaError_t wait_logits0(Ctx *c, cudaStream_t st)
{
    if (!c->l0_event || c->from_hidden) return cudaSuccess;
    return cudaStreamWaitEvent(st, c->l0_event, 0);
}

inline void prof_mark(Ctx *c, int mark, cudaStream_t st)
{
    if (!c->prof_enabled) return;
    cudaEventRecord(c->prof_events[(c->prof_calls % kProfSlots) * kProfMarks + mark], st);
    if (mark == kProfMarks - 1) c->prof_calls++;
}

// Programmatic dependent launch.  A kernel that calls pdl_wait() before it touches anything an
// earlier kernel of the stream wrote may be launched with launch_k(..., pdl = true): it is then
// scheduled while its predecessor drains instead of after it.  pdl_trigger() lets the kernel's
// own successor do the same.  Launched without the attribute both calls do nothing.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_k(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                            bool pdl, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// ---- CUDA-core kernel family (simt_kernels.cu) -------------------------------------
cudaError_t simt_draft(Ctx *c, const void *hidden, const float *logits0, const int32_t *row_index,
                       int M, int K, const mrp_draft_out &out, cudaStream_t st);

// Optional exact recomputation of each row-step's top logit during the combine (used when the
// LM-head operands were rounded to fp16): l_top = l_0[row, tok] + W_lm[tok] . (h_k - h_0) in
// fp32 from the bf16 hi + lo rows, which removes the dominant token's rounding error from
// log-sum-exp and confidence.  w == nullptr: off.
// Element i of the caller's base logits, stored as fp32 or (is_bf16) as bf16.
__device__ __forceinline__ float ld_l0(const float *l0, int is_bf16, size_t i)
{
    return is_bf16 ? __bfloat162float(__ldg(reinterpret_cast<const __nv_bfloat16 *>(l0) + i)) : __ldg(l0 + i);
}

struct TopFix {
    const __nv_bfloat16 *w;      // [V, d]; nullptr: no recomputation
    const __nv_bfloat16 *xt;     // hi rows [n_rs, d] of the stacked LM-head operand, row-step major, then (from
                                 // row n_rs on, only read when w is set) the lo rows; nullptr: nothing to check
    const float *logits0;
    const int32_t *row_index;
    int d, V, M, n_rs;
    int n_rows_in;               // row_index entries at or above are invalid (their l_0 reads as zero)
    int l0_bf16;                 // logits0 holds bf16 values
    float range_limit;           // > 0: raise MRP_DEV_RANGE for a row-step whose operand has d * rms above it
};

// A caller-provided row index is used as an address only if it lies inside the caller's array.
__device__ __forceinline__ bool row_ok(int idx, int n_rows_in) { return (unsigned)idx < (unsigned)n_rows_in; }

// Shared by both families: merge per-slice partials into conf/lse/token/margin.
cudaError_t launch_combine(Ctx *c, const Partial *partials, int n_slices, int n_rowsteps,
                           const mrp_draft_out &out, int32_t *status, cudaStream_t st,
                           const TopFix *fix = nullptr, int M = 0);
// Probability, under every step's logits, of the token on top at step 0 (mrp_draft_out.conf_first):
// l_k[tok_0] = l_0[row, tok_0] + W_lm[tok_0] . x_k exactly in fp32, then exp(l_k[tok_0] - lse_k).  Runs
// after the combine, which provides token and lse.  x: the stacked LM-head operand rows, either fp32
// (CUDA-core family: step k >= 1 at row (k-1)*M + m) or bf16 hi + lo (tensor-core family: row k*M + m, lo
// rows lo_rows further on).
struct FirstTok {
    const void *w;            // [V, d], fp32 or bf16, or (w8_scale set) e4m3 codes with one scale per row
    int w_bf16;
    const float *w8_scale;
    const float *logits0;     // nullptr: base logits computed in the pass (their operand rows are part of x)
    int l0_bf16;
    const int32_t *row_index;
    int n_rows_in;
    const void *x;
    int x_bf16;               // 0: fp32 rows, 1: bf16 hi + lo rows
    long long lo_rows;
    int M, K, d, V;
};
cudaError_t launch_first_token_prob(Ctx *c, const FirstTok &f, const mrp_draft_out &out, cudaStream_t st);

// CUDA-core family: gather masked rows of `hidden` into fp32 h0f / hcur (xt0: where the step-0
// operand rows n_0 go when the base logits are computed in the LM-head pass, else nullptr).
cudaError_t launch_prep(Ctx *c, const void *hidden, const int32_t *row_index, int M,
                        cudaStream_t st, float *xt0, int32_t *user_status);

// ---- selection / verification (select_verify.cu) ------------------------------------
cudaError_t launch_commit(Ctx *c, const mrp_select_out &sel, const int8_t *accept_mask, int B, int L, int Kd,
                          const mrp_block_state &state, cudaStream_t st);
cudaError_t launch_select(Ctx *c, const float *conf, const int32_t *token, const int32_t *row_index,
                          int M, int K, int B, int L, const mrp_select_params &p,
                          const mrp_select_out &out, cudaStream_t st);
cudaError_t launch_verify(Ctx *c, const int32_t *draft_tok, const int32_t *verify_tok,
                          const int32_t *draft_len, int B, int Kd, int positionwise,
                          int32_t *accept_len, int8_t *accept_mask, cudaStream_t st);

// Launches the bounded-wait self-test kernel (tc_kernels.cu).
cudaError_t tc_selftest_timeout(Ctx *c, int32_t *user_status, cudaStream_t st);

// ---- tensor-core kernel family (tc_*.cu) ---------------------------------------------
bool tc_supported(const mrp_config &cfg, const mrp_head_weights *heads, const void *w_lm);
cudaError_t tc_create(Ctx *c);
void tc_destroy(Ctx *c);
cudaError_t tc_draft(Ctx *c, const void *hidden, const float *logits0, const int32_t *row_index,
                     int M, int K, const mrp_draft_out &out, cudaStream_t st);

// Which kernels serve a call of M rows and K steps (tc_plan also sets the lo-block offsets lo_x / lo_xt of
// the context for the call), and the part of a drafting pass behind the head chain: LM head on the stacked
// operand rows already in the workspace (xt; xt16 in fp16 mode), combine, per-token probability.
struct TcPlan {
    bool pdl, few_rows, lm_few, f16_lm, chain, with_kl;
    int n_rs;
};
TcPlan tc_plan(Ctx *c, int M, int K, const mrp_draft_out &out, cudaStream_t st, bool want_chain);
cudaError_t tc_lm_tail(Ctx *c, const TcPlan &pl, const float *logits0, const int32_t *row_index, int M, int K,
                       const mrp_draft_out &out, cudaStream_t st);
// Row-major tensor-core products on operands of the caller's own (the module): see tc_kernels.cu.
cudaError_t tc_linear(Ctx *c, const __nv_bfloat16 *a, int n, int n_in, const void *w, int n_out, const float *sumsq,
                      int n_ss, float *out, bool accumulate, int32_t *user_status, cudaStream_t st, const void *gamma_next,
                      __nv_bfloat16 *xg_next, float *sumsq_out, int *n_ss_out);
cudaError_t tc_linear3(Ctx *c, const __nv_bfloat16 *a, int n, int n_in, const void *w0, const void *w1, const void *w2,
                       int n_out, const float *sumsq, int n_ss, float *out0, float *out1, float *out2, int32_t *user_status,
                       cudaStream_t st);
cudaError_t tc_gate_up(Ctx *c, const __nv_bfloat16 *a, int n, int n_in, const void *w_gate, const void *w_up, int F,
                       const float *sumsq, int n_ss, __nv_bfloat16 *act, int32_t *user_status, cudaStream_t st);
// Few-row tensor-core products on the caller's own operands (n <= 64 rows; lo rows sk_head_pad(n) rows behind the
// hi rows): see tc_skinny.cu.
cudaError_t sk_linear(Ctx *c, const __nv_bfloat16 *a, int n, int n_in, const void *w, int n_out, const float *sumsq,
                      int n_ss, float *out, bool accumulate, const void *gamma_next, __nv_bfloat16 *xg_next,
                      float *sumsq_out, int *n_ss_out, int32_t *user_status, cudaStream_t st);
cudaError_t sk_linear3(Ctx *c, const __nv_bfloat16 *a, int n, int n_in, const void *w0, const void *w1, const void *w2,
                       int n_out, const float *sumsq, int n_ss, float *out0, float *out1, float *out2, int32_t *user_status,
                       cudaStream_t st);
cudaError_t sk_gate_up(Ctx *c, const __nv_bfloat16 *a, int n, int n_in, const void *w_gate, const void *w_up, int F,
                       const float *sumsq, int n_ss, __nv_bfloat16 *act, int32_t *user_status, cudaStream_t st);
// One module step as one cooperative kernel (see tc_chain.cu); bar_mem: kModChainBarInts zero-able ints.
constexpr int kModChainBarInts = 22 * 448 + 1;
cudaError_t sk_module_step(Ctx *c, int n, int L, const int32_t *tokens, const void *hidden0, float *h_state, bool first_step,
                           __nv_bfloat16 *cat16, __nv_bfloat16 *xa, __nv_bfloat16 *xb, __nv_bfloat16 *act16, float *q, float *k,
                           float *v, float *z, int32_t *bar_mem, const int32_t *row_index, int n_masked, int lo_xt, bool f16_lm,
                           float *hidden_out, int32_t *user_status, cudaStream_t st, bool check_only, float *att_part = nullptr,
                           int *att_counters = nullptr);
// The same for the CUDA-core family (operand rows: fp32 xt).
cudaError_t simt_lm_tail(Ctx *c, const float *logits0, const int32_t *row_index, int M, int K,
                         const mrp_draft_out &out, cudaStream_t st);

// One step of the token-conditioned module (simt_kernels.cu): module forward on CUDA cores, then the
// context's LM-head tail.
cudaError_t module_step(Ctx *c, const int32_t *tokens, const void *hidden0, float *h_state, const float *logits0,
                        const int32_t *row_index, int M, int B, int L, bool first_step, const mrp_draft_out &out,
                        cudaStream_t st);
size_t module_workspace_bytes(const mrp_config &cfg, int n_layers);
size_t module_att_offset(const mrp_config &cfg);   // the clean-prefix attention's area of the module workspace

// Few-row variants (tc_skinny.cu): weight rows on the MMA M axis; rows <= 32.
bool sk_rows_ok(int rows);          // LM head: row-steps incl. step 0
bool sk_head_rows_ok(int M);       // head chain: masked rows
int sk_head_pad(int M);            // rows of an activation block as the few-row head kernels see it
int sk_lm_pad(int n_rs);           // likewise for the few-row LM-head kernel
cudaError_t sk_gateup(Ctx *c, int k, int M, int K, int n_ss, const mrp_draft_out &out, cudaStream_t st, bool pdl);
cudaError_t sk_down(Ctx *c, int k, int M, int K, const mrp_draft_out &out, cudaStream_t st, bool pdl,
                    int *n_ss_out, bool f16_lm);
bool sk_heads_ok(const mrp_config &cfg);
// The whole head chain as one cooperative kernel (tc_chain.cu); cudaErrorNotSupported = use the others.
cudaError_t sk_chain(Ctx *c, int M, int K, const mrp_draft_out &out, cudaStream_t st, bool f16_lm,
                     bool check_only);
cudaError_t sk_lm(Ctx *c, const float *logits0, const int32_t *row_index, int M, int K,
                  const mrp_draft_out &out, cudaStream_t st, bool pdl);
bool fp8_lm_supported(const mrp_config &cfg);
cudaError_t fp8_lm_create(Ctx *c);      // quantises W_lm into the workspace (blocking, once)

__device__ inline KlPartial merge_kl(const KlPartial &a, const KlPartial &b)
{
    KlPartial r;
    r.mx = fmaxf(a.mx, b.mx);
    const float ea = (a.sum == 0.f) ? 0.f : expf(a.mx - r.mx), eb = (b.sum == 0.f) ? 0.f : expf(b.mx - r.mx);
    r.sum = a.sum * ea + b.sum * eb;
    r.cross = a.cross * ea + b.cross * eb;
    r.pad = 0.f;
    return r;
}

// Merge of two partial statistics; ties on the maximum go to the lower token id.
__device__ inline Partial merge_partial(const Partial &a, const Partial &b)
{
    Partial r;
    const bool b_wins = (b.mx > a.mx) || (b.mx == a.mx && b.idx < a.idx);
    const float hi = b_wins ? b.mx : a.mx;
    const float lo = b_wins ? a.mx : b.mx;
    r.mx = hi;
    r.idx = b_wins ? b.idx : a.idx;
    float sec = lo;
    sec = a.second > sec ? a.second : sec;
    sec = b.second > sec ? b.second : sec;
    r.second = sec;
    const float ea = (a.sum == 0.f) ? 0.f : a.sum * expf(a.mx - hi);
    const float eb = (b.sum == 0.f) ? 0.f : b.sum * expf(b.mx - hi);
    r.sum = ea + eb;
    return r;
}

// ---- the module's attention behind a clean prefix (Fig. 1(c)) ------------------------------------------------
// Work unit = (block b, attention head, chunk of the key range), run by the four warps of a CTA (or of its epilogue
// warpgroup).  Keys and values: the first P rows of the (sequence, head) slab of the prefix cache (type T, written by
// earlier calls, read through the read-only path), then the L rows of the block (fp32, possibly written earlier in
// this same kernel: read from L2).  The keys go in groups of 32 (prefix groups, then block groups); chunk ch covers
// groups [ch * gpc, (ch + 1) * gpc) and its warps take them round-robin: a lane per key for the scores of kAttQT
// queries at a time (a key row is loaded once for all of them), then lanes over the head's features for the weighted
// values, with a running maximum and sum per query.  The four warps' partial results meet in shared memory; with
// more than one chunk the chunk's partial results go to `part` and the CTA that arrives last at the (block, head)
// counter merges them -- no CTA waits for another.
//   q, kb, vb   the block's first row of q / k / v at the head's columns, row stride d; pk, pv the first row of the
//               (sequence, head) slab of the cache, whose rows are the head's dh features, one after the other
//   part        [n_ch][L][dh + 2] floats of this (block, head); counter: its arrival counter, zero before and after
//   sh          att_sh_floats(dh) floats of shared memory, 16-byte aligned;  sync(): a barrier over exactly these
//               128 threads;  out(i, c, value) is called once per query i of the block and feature c of the head
constexpr int kAttMaxDh = 256;
constexpr int kAttQT = 4;
constexpr int kAttMaxChunks = 32;                      // (the merge puts a lane on every chunk)
constexpr int kAttCounters = 4096;                    // (block, head) pairs that can split their keys over CTAs
constexpr size_t kAttPartFloats = (size_t)1 << 20;    // partial results of split units
__host__ __device__ constexpr int att_sh_floats(int dh) { return kAttQT * dh + 4 * kAttQT * (dh + 2); }

// How a call splits the keys: groups per chunk and chunks, for sequences of up to `cap` prefix rows and blocks of L,
// aiming at `target` units in all.
struct AttSplit { int gpc, n_ch; };
inline AttSplit att_split(int cap, int L, int BH, int dh, int target)
{
    const int groups = (cap + 31) / 32 + (L + 31) / 32;
    int want = BH > 0 ? target / BH : 1;
    if (want > kAttMaxChunks) want = kAttMaxChunks;
    if (want > groups) want = groups;
    const size_t per_chunk = (size_t)BH * L * (dh + 2);
    if (BH > kAttCounters || per_chunk > kAttPartFloats) want = 1;
    else if ((size_t)want * per_chunk > kAttPartFloats) want = (int)(kAttPartFloats / per_chunk);
    if (want < 1) want = 1;
    AttSplit sp;
    sp.gpc = (groups + want - 1) / want;
    sp.n_ch = (groups + sp.gpc - 1) / sp.gpc;
    return sp;
}

__device__ __forceinline__ float att_f(float x) { return x; }
__device__ __forceinline__ float att_f(__nv_bfloat16 x) { return __bfloat162float(x); }

// eight consecutive elements of a row as floats (16-byte aligned); CG: through L2 (data written in this kernel)
template <bool CG>
__device__ __forceinline__ void att_ld8(const __nv_bfloat16 *p, float f[8])
{
    const uint4 u = __ldg(reinterpret_cast<const uint4 *>(p));
    const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&u);
#pragma unroll
    for (int x = 0; x < 4; ++x) {
        const float2 t = __bfloat1622float2(h[x]);
        f[2 * x] = t.x;
        f[2 * x + 1] = t.y;
    }
}
template <bool CG>
__device__ __forceinline__ void att_ld8(const float *p, float f[8])
{
    const float4 *p4 = reinterpret_cast<const float4 *>(p);
    const float4 a = CG ? __ldcg(p4) : __ldg(p4), b = CG ? __ldcg(p4 + 1) : __ldg(p4 + 1);
    f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
}
template <bool CG, typename T>
__device__ __forceinline__ float att_ld1(const T *p)
{
    if (CG) return att_f(__ldcg(p));
    return att_f(__ldg(p));
}

// scores of one key row against the kAttQT staged queries (q_s: [kAttQT][dh])
template <bool CG, typename T>
__device__ __forceinline__ void att_scores(const float *q_s, const T *row, int dh, bool vec, float s[kAttQT])
{
#pragma unroll
    for (int qi = 0; qi < kAttQT; ++qi) s[qi] = 0.f;
    if (vec && (dh & 31) == 0) {
        // 32 elements of the row per step: four loads in flight together, several steps overlapping
#pragma unroll 4
        for (int c = 0; c < dh; c += 32) {
            float f[4][8];
#pragma unroll
            for (int x = 0; x < 4; ++x) att_ld8<CG>(row + c + 8 * x, f[x]);
#pragma unroll
            for (int qi = 0; qi < kAttQT; ++qi) {
                const float *qq = q_s + qi * dh + c;
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                    const float4 a = *reinterpret_cast<const float4 *>(qq + 8 * x), b = *reinterpret_cast<const float4 *>(qq + 8 * x + 4);
                    s[qi] = fmaf(a.x, f[x][0], s[qi]); s[qi] = fmaf(a.y, f[x][1], s[qi]);
                    s[qi] = fmaf(a.z, f[x][2], s[qi]); s[qi] = fmaf(a.w, f[x][3], s[qi]);
                    s[qi] = fmaf(b.x, f[x][4], s[qi]); s[qi] = fmaf(b.y, f[x][5], s[qi]);
                    s[qi] = fmaf(b.z, f[x][6], s[qi]); s[qi] = fmaf(b.w, f[x][7], s[qi]);
                }
            }
        }
    } else if (vec) {
        for (int c = 0; c < dh; c += 8) {
            float f[8];
            att_ld8<CG>(row + c, f);
#pragma unroll
            for (int qi = 0; qi < kAttQT; ++qi)
#pragma unroll
                for (int x = 0; x < 8; ++x) s[qi] = fmaf(q_s[qi * dh + c + x], f[x], s[qi]);
        }
    } else {
        for (int c = 0; c < dh; ++c) {
            const float f = att_ld1<CG>(row + c);
#pragma unroll
            for (int qi = 0; qi < kAttQT; ++qi) s[qi] = fmaf(q_s[qi * dh + c], f, s[qi]);
        }
    }
}

// the lane's features of a value row: PER consecutive ones from lane * PER (PER > 0), or lane + 32 u, u < 8 (PER == 0)
template <int PER, bool CG, typename T>
__device__ __forceinline__ void att_ldv(const T *row, int lane, int dh, float v[8])
{
    if (PER == 8) {
        att_ld8<CG>(row + lane * 8, v);
    } else if (PER == 4 && sizeof(T) == 2) {
        const uint2 u = __ldg(reinterpret_cast<const uint2 *>(row + lane * 4));
        const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&u);
        const float2 a = __bfloat1622float2(h[0]), b = __bfloat1622float2(h[1]);
        v[0] = a.x; v[1] = a.y; v[2] = b.x; v[3] = b.y;
    } else if (PER == 4) {
        const float4 *p4 = reinterpret_cast<const float4 *>(row + lane * 4);
        const float4 a = CG ? __ldcg(p4) : __ldg(p4);
        v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
    } else if (PER > 0) {
#pragma unroll
        for (int u = 0; u < PER; ++u) v[u] = att_ld1<CG>(row + lane * PER + u);
    } else {
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = lane + 32 * u < dh ? att_ld1<CG>(row + lane + 32 * u) : 0.f;
    }
}

// one group of up to 32 keys (rows krow0 + j * d, vrow0 + j * d, j < cnt) folded into the warp's running state
template <int PER, bool CG, typename T>
__device__ __forceinline__ void att_group(const float *q_s, const T *krow0, const T *vrow0, int cnt, int d, int dh, bool vec, float scale,
                                          int lane, float mx[kAttQT], float sum[kAttQT], float (&oacc)[kAttQT][8])
{
    constexpr int NU = PER > 0 ? PER : 8;
    float s[kAttQT], pj[kAttQT];
    if (lane < cnt) {
        att_scores<CG>(q_s, krow0 + (size_t)lane * d, dh, vec, s);
    } else {
#pragma unroll
        for (int qi = 0; qi < kAttQT; ++qi) s[qi] = -INFINITY;
    }
#pragma unroll
    for (int qi = 0; qi < kAttQT; ++qi) {
        s[qi] *= scale;
        float gm = s[qi];
#pragma unroll
        for (int w = 16; w > 0; w >>= 1) gm = fmaxf(gm, __shfl_xor_sync(0xffffffffu, gm, w));
        const float nm = fmaxf(mx[qi], gm), corr = expf(mx[qi] - nm);       // (first group: mx = -inf, corr = 0)
        pj[qi] = lane < cnt ? expf(s[qi] - nm) : 0.f;
        sum[qi] = sum[qi] * corr + pj[qi];                                   // per-lane share; corr is the same in every lane
#pragma unroll
        for (int u = 0; u < NU; ++u) oacc[qi][u] *= corr;
        mx[qi] = nm;
    }
    // weighted values: eight or sixteen keys' rows in flight together; a key index beyond the group reads the group's last row
    // with weight 0 (the lanes beyond cnt hold pj = 0)
    constexpr int VB = NU <= 4 ? 16 : 8;
    for (int j0 = 0; j0 < cnt; j0 += VB) {
        float v[VB][8];
#pragma unroll
        for (int x = 0; x < VB; ++x) {
            const int j = j0 + x < cnt ? j0 + x : cnt - 1;
            att_ldv<PER, CG>(vrow0 + (size_t)j * d, lane, dh, v[x]);
        }
#pragma unroll
        for (int x = 0; x < VB; ++x)
#pragma unroll
            for (int qi = 0; qi < kAttQT; ++qi) {
                const float w = __shfl_sync(0xffffffffu, pj[qi], (j0 + x) & 31);
#pragma unroll
                for (int u = 0; u < NU; ++u) oacc[qi][u] = fmaf(w, v[x][u], oacc[qi][u]);
            }
    }
}

// The chunks of a (block, head) meet: every CTA arrives at the pair's counter once its partial results are written;
// the CTA that arrives last merges them (a warp per query) and leaves the counter at zero.  No CTA waits.
template <typename Sync, typename Out>
__device__ __forceinline__ void att_arrive_merge(int n_ch, int L, int dh, float *part, int *counter, float *sh, int warp, int lane,
                                                 Sync sync, Out out)
{
    const int t = warp * 32 + lane, stride = dh + 2;
    {
        // arrive at the (block, head) counter; the CTA that arrives last merges the chunks and leaves the counter at zero
        int *flag = reinterpret_cast<int *>(sh);
        __threadfence();
        sync();
        if (t == 0) {
            const int old = atomicAdd(counter, 1);
            *flag = old == n_ch - 1;
            if (old == n_ch - 1) {
                __threadfence();
                *counter = 0;
            }
        }
        sync();
        const bool last = *flag != 0;
        sync();
        if (last) {
            // a warp per query: lanes over the chunks for the weights, then over the features, the partial results of
            // all chunks in flight together
            for (int i = warp; i < L; i += 4) {
                const float m = lane < n_ch ? __ldcg(part + ((size_t)lane * L + i) * stride) : -INFINITY;
                const float sm = lane < n_ch ? __ldcg(part + ((size_t)lane * L + i) * stride + 1) : 0.f;
                float top = m;
#pragma unroll
                for (int w = 16; w > 0; w >>= 1) top = fmaxf(top, __shfl_xor_sync(0xffffffffu, top, w));
                const float e = m == -INFINITY ? 0.f : expf(m - top);
                float tot = sm * e;
#pragma unroll
                for (int w = 16; w > 0; w >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, w);
                float o[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) o[u] = 0.f;
#pragma unroll 4
                for (int x = 0; x < n_ch; ++x) {
                    const float ex = __shfl_sync(0xffffffffu, e, x);
                    const float *src = part + ((size_t)x * L + i) * stride + 2;
#pragma unroll
                    for (int u = 0; u < 8; ++u)
                        if (lane + 32 * u < dh) o[u] = fmaf(__ldcg(src + lane + 32 * u), ex, o[u]);
                }
#pragma unroll
                for (int u = 0; u < 8; ++u)
                    if (lane + 32 * u < dh) out(i, lane + 32 * u, o[u] / tot);
            }
        }
    }
}

template <int PER, typename T, typename Sync, typename Out>
__device__ __forceinline__ void att_unit_per(const float *q, const T *pk, const T *pv, int P, const float *kb, const float *vb, int L,
                                             int d, int dh, int g_lo, int g_hi, int ch, int n_ch, float *part, int *counter, float *sh,
                                             int warp, int lane, Sync sync, Out out)
{
    // (groups [g_lo, g_hi) of the sequence's prefix groups followed by its block groups; ch: the slot of the partial results)
    constexpr int NU = PER > 0 ? PER : 8;
    float *q_s = sh, *part_s = sh + kAttQT * dh;              // part_s[w][qi]: maximum, sum, o[dh]
    const int t = warp * 32 + lane, stride = dh + 2;
    const float scale = rsqrtf((float)dh);
    const bool vec = (dh % 8) == 0 && (d % 8) == 0;
    const int gp = (P + 31) / 32, gb = (L + 31) / 32;
    const int g_end = g_hi < gp + gb ? g_hi : gp + gb;
    auto feat = [&](int u) { return PER > 0 ? lane * PER + u : lane + 32 * u; };
    // The prefix rows this warp will read, asked into L2 up front: each lane reads whole rows of its own in the score
    // loops, a handful of loads at a time, and would otherwise pay the DRAM latency once per handful.
    for (int g = g_lo + warp; g < g_end && g < gp; g += 4) {
        const int j = g * 32 + lane;
        if (j < P) {
            const char *rk = reinterpret_cast<const char *>(pk + (size_t)j * dh), *rv = reinterpret_cast<const char *>(pv + (size_t)j * dh);
            for (int off = 0; off < dh * (int)sizeof(T); off += 128) {
                asm volatile("prefetch.global.L2 [%0];" ::"l"(rk + off));
                asm volatile("prefetch.global.L2 [%0];" ::"l"(rv + off));
            }
        }
    }
    for (int q0 = 0; q0 < L; q0 += kAttQT) {
        // the tile's queries (zero rows beyond the block)
        for (int x = t; x < kAttQT * dh; x += 128) {
            const int qi = x / dh, c = x - qi * dh;
            q_s[x] = q0 + qi < L ? __ldcg(q + (size_t)(q0 + qi) * d + c) : 0.f;
        }
        sync();
        float mx[kAttQT], sum[kAttQT], oacc[kAttQT][8];
#pragma unroll
        for (int qi = 0; qi < kAttQT; ++qi) {
            mx[qi] = -INFINITY;
            sum[qi] = 0.f;
#pragma unroll
            for (int u = 0; u < 8; ++u) oacc[qi][u] = 0.f;
        }
        for (int g = g_lo + warp; g < g_end; g += 4) {
            if (g < gp) {
                const int j0 = g * 32, left = P - j0;
                att_group<PER, false>(q_s, pk + (size_t)j0 * dh, pv + (size_t)j0 * dh, left < 32 ? left : 32, dh, dh, vec, scale, lane, mx, sum,
                                      oacc);
            } else {
                const int j0 = (g - gp) * 32, left = L - j0;
                att_group<PER, true>(q_s, kb + (size_t)j0 * d, vb + (size_t)j0 * d, left < 32 ? left : 32, d, dh, vec, scale, lane, mx, sum,
                                     oacc);
            }
        }
#pragma unroll
        for (int qi = 0; qi < kAttQT; ++qi) {
            float sm = sum[qi];
#pragma unroll
            for (int w = 16; w > 0; w >>= 1) sm += __shfl_xor_sync(0xffffffffu, sm, w);
            float *mine = part_s + (size_t)(warp * kAttQT + qi) * stride;
            if (lane == 0) {
                mine[0] = mx[qi];
                mine[1] = sm;
            }
#pragma unroll
            for (int u = 0; u < NU; ++u)
                if (feat(u) < dh) mine[2 + feat(u)] = oacc[qi][u];
        }
        sync();
        // the four warps' results of each query of the tile: merged, and either final or this chunk's partial result
        for (int qi = 0; qi < kAttQT && q0 + qi < L; ++qi) {
            float top = -INFINITY, e[4], tot = 0.f;
#pragma unroll
            for (int w = 0; w < 4; ++w) top = fmaxf(top, part_s[(size_t)(w * kAttQT + qi) * stride]);
#pragma unroll
            for (int w = 0; w < 4; ++w) {
                const float m = part_s[(size_t)(w * kAttQT + qi) * stride];
                e[w] = m == -INFINITY ? 0.f : expf(m - top);          // (a warp, or a whole chunk, without keys)
                tot = fmaf(part_s[(size_t)(w * kAttQT + qi) * stride + 1], e[w], tot);
            }
            float *dst = part + ((size_t)ch * L + q0 + qi) * stride;
            if (n_ch > 1 && t == 0) {
                dst[0] = top;
                dst[1] = tot;
            }
            for (int c = t; c < dh; c += 128) {
                float o = 0.f;
#pragma unroll
                for (int w = 0; w < 4; ++w) o = fmaf(part_s[(size_t)(w * kAttQT + qi) * stride + 2 + c], e[w], o);
                if (n_ch > 1) dst[2 + c] = o;
                else out(q0 + qi, c, o / tot);
            }
        }
        sync();                                               // sh is free again
    }
    if (n_ch > 1) att_arrive_merge(n_ch, L, dh, part, counter, sh, warp, lane, sync, out);
}

// ---- the prefix part on tensor cores ------------------------------------------------------------------------
// For bf16 caches and heads of 64 or 128 features the prefix groups of a chunk run as small matrix products
// (mma.sync m16n8k16, bf16 operands, fp32 accumulation): S = Q K^T over 16 queries x 32 keys per group, online softmax on
// the accumulator fragments, O += P V.  Queries and probabilities enter as bf16 hi + lo pairs (two products each), keys
// and values are the cache's own bf16.  The contraction index of S runs over features in an order that lets every
// lane fetch 16 bytes of a key row at once (A and B use the same order, so the sum is the same); the value rows are
// fetched the same way and turned with movmatrix, which leaves each lane with eight consecutive features of two
// queries.  Only cache rows pass through here: the block's own fp32 keys and values are a chunk of their own on the
// CUDA-core routine above, and the chunks always meet through att_arrive_merge.
__device__ __forceinline__ void att_mma16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t att_movm(uint32_t a)
{
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
// (x, y) as a bf16 pair, x in the low half; and the pair of what that rounding left over
__device__ __forceinline__ void att_split2(float x, float y, uint32_t &hi, uint32_t &lo)
{
    const __nv_bfloat162 h = __floats2bfloat162_rn(x, y);
    const float2 hf = __bfloat1622float2(h);
    const __nv_bfloat162 l = __floats2bfloat162_rn(x - hf.x, y - hf.y);
    hi = *reinterpret_cast<const uint32_t *>(&h);
    lo = *reinterpret_cast<const uint32_t *>(&l);
}
__device__ __forceinline__ uint32_t att_comp(const uint4 &v, int i) { return i == 0 ? v.x : i == 1 ? v.y : i == 2 ? v.z : v.w; }

// shared floats the tensor-core unit needs: 16 staged queries as bf16 hi + lo rows (padded), or the merge area
__host__ __device__ constexpr int att_mma_sh_floats(int dh)
{
    return (2 * 16 * (dh + 8)) / 2 > 4 * 4 * (dh + 2) ? (2 * 16 * (dh + 8)) / 2 : 4 * 4 * (dh + 2);
}

template <int NG, typename Sync>
__device__ __forceinline__ void att_unit_mma(const float *q, const __nv_bfloat16 *pk, const __nv_bfloat16 *pv, int P, int L, int d, int g_lo,
                                             int g_hi, float *part_slot, float *sh, int warp, int lane, Sync sync)
{
    constexpr int DH = 32 * NG, QS = DH + 8, stride = DH + 2;
    __nv_bfloat16 *q_hi = reinterpret_cast<__nv_bfloat16 *>(sh), *q_lo = q_hi + 16 * QS;
    float *part_s = sh;                                   // [4 warps][4 queries][DH + 2], once the queries are done with
    const int t = warp * 32 + lane, r = lane >> 2, j = lane & 3;
    const float scale = rsqrtf((float)DH);
    const int gp = (P + 31) / 32;
    if (g_hi > gp) g_hi = gp;
    if (g_lo < g_hi) {
        // the chunk's rows (one contiguous run per tensor in the head-major cache) asked into L2 up front: a group then
        // pays the L2 latency three times (keys, two halves of the values), not the DRAM latency
        const int row_hi = g_hi * 32 < P ? g_hi * 32 : P;
        const char *k0 = reinterpret_cast<const char *>(pk + (size_t)g_lo * 32 * DH), *v0 = reinterpret_cast<const char *>(pv + (size_t)g_lo * 32 * DH);
        const size_t bytes = (size_t)(row_hi - g_lo * 32) * DH * 2;
        for (size_t off = (size_t)t * 128; off < bytes; off += 128 * 128) {
            asm volatile("prefetch.global.L2 [%0];" ::"l"(k0 + off));
            asm volatile("prefetch.global.L2 [%0];" ::"l"(v0 + off));
        }
    }
    for (int q0 = 0; q0 < L; q0 += 16) {
        const int nq = L - q0 < 16 ? L - q0 : 16;
        for (int x = t; x < 16 * DH; x += 128) {
            const int qi = x / DH, c = x - qi * DH;
            const float v = qi < nq ? __ldcg(q + (size_t)(q0 + qi) * d + c) : 0.f;
            const __nv_bfloat16 h = __float2bfloat16_rn(v);
            q_hi[qi * QS + c] = h;
            q_lo[qi * QS + c] = __float2bfloat16_rn(v - __bfloat162float(h));
        }
        sync();
        float o[NG][4][4];
#pragma unroll
        for (int a = 0; a < NG; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b)
#pragma unroll
                for (int c = 0; c < 4; ++c) o[a][b][c] = 0.f;
        float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;      // rows r and r + 8 of the tile
        for (int g = g_lo + warp; g < g_hi; g += 4) {
            const int j0 = g * 32, left = P - j0, cnt = left < 32 ? left : 32;
            // ---- S = Q K^T: four tiles of 8 keys; a key index beyond the group reads the group's last row (masked below)
            float sacc[4][4];
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) sacc[a][b] = 0.f;
            // the value rows of the first 16 keys are asked for together with the keys: one round of loads less
            uint4 va0[NG], vb0[NG];
            {
                const int k0 = r < cnt ? r : cnt - 1, k1 = 8 + r < cnt ? 8 + r : cnt - 1;
#pragma unroll
                for (int a = 0; a < NG; ++a) {
                    va0[a] = __ldg(reinterpret_cast<const uint4 *>(pv + (size_t)(j0 + k0) * DH + 32 * a + 8 * j));
                    vb0[a] = __ldg(reinterpret_cast<const uint4 *>(pv + (size_t)(j0 + k1) * DH + 32 * a + 8 * j));
                }
            }
            // every key row piece of the group in flight at once (the products below would otherwise wait for them
            // one 32-feature step at a time)
            uint4 kall[NG][4];
#pragma unroll
            for (int tt = 0; tt < 4; ++tt) {
                const int key = 8 * tt + r < cnt ? 8 * tt + r : cnt - 1;
#pragma unroll
                for (int s = 0; s < NG; ++s)
                    kall[s][tt] = __ldg(reinterpret_cast<const uint4 *>(pk + (size_t)(j0 + key) * DH + 32 * s + 8 * j));
            }
#pragma unroll
            for (int s = 0; s < NG; ++s) {
                const uint4 *kk = kall[s];
                const uint4 ah0 = *reinterpret_cast<const uint4 *>(q_hi + r * QS + 32 * s + 8 * j);
                const uint4 ah1 = *reinterpret_cast<const uint4 *>(q_hi + (r + 8) * QS + 32 * s + 8 * j);
                const uint4 al0 = *reinterpret_cast<const uint4 *>(q_lo + r * QS + 32 * s + 8 * j);
                const uint4 al1 = *reinterpret_cast<const uint4 *>(q_lo + (r + 8) * QS + 32 * s + 8 * j);
#pragma unroll
                for (int tt = 0; tt < 4; ++tt) {
                    att_mma16816(sacc[tt], ah0.x, ah1.x, ah0.y, ah1.y, kk[tt].x, kk[tt].y);
                    att_mma16816(sacc[tt], al0.x, al1.x, al0.y, al1.y, kk[tt].x, kk[tt].y);
                    att_mma16816(sacc[tt], ah0.z, ah1.z, ah0.w, ah1.w, kk[tt].z, kk[tt].w);
                    att_mma16816(sacc[tt], al0.z, al1.z, al0.w, al1.w, kk[tt].z, kk[tt].w);
                }
            }
            // ---- online softmax on the fragments: [0], [1] belong to row r, [2], [3] to row r + 8; columns = keys 8 tt + 2 j + e
            float g0 = -INFINITY, g1 = -INFINITY;
#pragma unroll
            for (int tt = 0; tt < 4; ++tt)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const bool in = 8 * tt + 2 * j + e < cnt;
                    sacc[tt][e] = in ? sacc[tt][e] * scale : -INFINITY;
                    sacc[tt][2 + e] = in ? sacc[tt][2 + e] * scale : -INFINITY;
                    g0 = fmaxf(g0, sacc[tt][e]);
                    g1 = fmaxf(g1, sacc[tt][2 + e]);
                }
            g0 = fmaxf(g0, __shfl_xor_sync(0xffffffffu, g0, 1));
            g0 = fmaxf(g0, __shfl_xor_sync(0xffffffffu, g0, 2));
            g1 = fmaxf(g1, __shfl_xor_sync(0xffffffffu, g1, 1));
            g1 = fmaxf(g1, __shfl_xor_sync(0xffffffffu, g1, 2));
            const float n0 = fmaxf(m0, g0), n1 = fmaxf(m1, g1);          // finite: the group has a key
            const float c0 = expf(m0 - n0), c1 = expf(m1 - n1);          // (first group: exp(-inf) = 0)
            float ps0 = 0.f, ps1 = 0.f;
#pragma unroll
            for (int tt = 0; tt < 4; ++tt)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    sacc[tt][e] = expf(sacc[tt][e] - n0);                // a masked key: exp(-inf) = 0
                    sacc[tt][2 + e] = expf(sacc[tt][2 + e] - n1);
                    ps0 += sacc[tt][e];
                    ps1 += sacc[tt][2 + e];
                }
            l0 = l0 * c0 + ps0;                                          // (the lane's share of the row sums)
            l1 = l1 * c1 + ps1;
            m0 = n0;
            m1 = n1;
#pragma unroll
            for (int a = 0; a < NG; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    o[a][b][0] *= c0; o[a][b][1] *= c0;
                    o[a][b][2] *= c1; o[a][b][3] *= c1;
                }
            // ---- O += P V: two steps of 16 keys; the probabilities as A fragments (hi + lo), the values turned by movmatrix
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                uint32_t ph[4], pl[4];
                att_split2(sacc[2 * u][0], sacc[2 * u][1], ph[0], pl[0]);
                att_split2(sacc[2 * u][2], sacc[2 * u][3], ph[1], pl[1]);
                att_split2(sacc[2 * u + 1][0], sacc[2 * u + 1][1], ph[2], pl[2]);
                att_split2(sacc[2 * u + 1][2], sacc[2 * u + 1][3], ph[3], pl[3]);
                const int k0 = 16 * u + r < cnt ? 16 * u + r : cnt - 1, k1 = 16 * u + 8 + r < cnt ? 16 * u + 8 + r : cnt - 1;
                uint4 va[NG], vb[NG];
#pragma unroll
                for (int a = 0; a < NG; ++a) {
                    if (u == 0) {
                        va[a] = va0[a];
                        vb[a] = vb0[a];
                    } else {
                        va[a] = __ldg(reinterpret_cast<const uint4 *>(pv + (size_t)(j0 + k0) * DH + 32 * a + 8 * j));
                        vb[a] = __ldg(reinterpret_cast<const uint4 *>(pv + (size_t)(j0 + k1) * DH + 32 * a + 8 * j));
                    }
                }
#pragma unroll
                for (int a = 0; a < NG; ++a)
#pragma unroll
                    for (int b = 0; b < 4; ++b) {
                        const uint32_t b0 = att_movm(att_comp(va[a], b)), b1 = att_movm(att_comp(vb[a], b));
                        att_mma16816(o[a][b], ph[0], ph[1], ph[2], ph[3], b0, b1);
                        att_mma16816(o[a][b], pl[0], pl[1], pl[2], pl[3], b0, b1);
                    }
            }
        }
        l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
        l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
        l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
        l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
        sync();                                              // the staged queries are done with: the merge area takes their place
        // the four warps' results, four queries at a time: rows 4 sub .. 4 sub + 3 sit in the lanes with r in
        // [4 (sub & 1), + 4), in fragment entries [0], [1] (sub < 2) or [2], [3]
#pragma unroll
        for (int sub = 0; sub < 4; ++sub) {
            if (4 * sub < nq) {
                const int rr = r - 4 * (sub & 1);
                if (rr >= 0 && rr < 4) {
                    float *mine = part_s + (size_t)(warp * 4 + rr) * stride;
                    if (j == 0) {
                        mine[0] = sub < 2 ? m0 : m1;
                        mine[1] = sub < 2 ? l0 : l1;
                    }
#pragma unroll
                    for (int a = 0; a < NG; ++a)
#pragma unroll
                        for (int b = 0; b < 4; ++b) {
                            mine[2 + 32 * a + 8 * j + 2 * b] = o[a][b][sub < 2 ? 0 : 2];
                            mine[2 + 32 * a + 8 * j + 2 * b + 1] = o[a][b][sub < 2 ? 1 : 3];
                        }
                }
                sync();
                for (int qi = 0; qi < 4 && 4 * sub + qi < nq; ++qi) {
                    float top = -INFINITY, e[4], tot = 0.f;
#pragma unroll
                    for (int w = 0; w < 4; ++w) top = fmaxf(top, part_s[(size_t)(w * 4 + qi) * stride]);
#pragma unroll
                    for (int w = 0; w < 4; ++w) {
                        const float m = part_s[(size_t)(w * 4 + qi) * stride];
                        e[w] = m == -INFINITY ? 0.f : expf(m - top);
                        tot = fmaf(part_s[(size_t)(w * 4 + qi) * stride + 1], e[w], tot);
                    }
                    float *dst = part_slot + (size_t)(q0 + 4 * sub + qi) * stride;
                    if (t == 0) {
                        dst[0] = top;
                        dst[1] = tot;
                    }
                    for (int c = t; c < DH; c += 128) {
                        float acc = 0.f;
#pragma unroll
                        for (int w = 0; w < 4; ++w) acc = fmaf(part_s[(size_t)(w * 4 + qi) * stride + 2 + c], e[w], acc);
                        dst[2 + c] = acc;
                    }
                }
                sync();
            }
        }
    }
}

// How a call on the tensor-core routine splits its keys: n_pre chunks of gpc prefix groups each, then the block's chunk.
inline AttSplit att_split_mma(int cap, int L, int BH, int dh, int target)
{
    const int groups = (cap + 31) / 32;
    int want = BH > 0 ? target / BH - 1 : 1;
    if (want > kAttMaxChunks - 1) want = kAttMaxChunks - 1;
    if (want > groups) want = groups;
    if (want < 1) want = 1;
    const size_t per_chunk = (size_t)BH * L * (dh + 2);
    while (want > 1 && (size_t)(want + 1) * per_chunk > kAttPartFloats) --want;
    AttSplit sp;
    sp.gpc = (groups + want - 1) / want;
    sp.n_ch = (groups + sp.gpc - 1) / sp.gpc + 1;
    return sp;
}
// Whether a call can use it (the caches are bf16: a tensor-core context).
inline bool att_mma_ok(int cap, int L, int BH, int d, int dh, const void *const *ptrs, int n_ptrs)
{
    if (cap < 1 || (dh != 64 && dh != 128) || (d % 8) || BH > kAttCounters) return false;
    if ((size_t)2 * BH * L * (dh + 2) > kAttPartFloats) return false;
    for (int i = 0; i < n_ptrs; ++i)
        if (reinterpret_cast<uintptr_t>(ptrs[i]) & 15u) return false;
    return true;
}

// (MMA: whether the kernel carries the tensor-core routine at all: it costs registers)
template <typename T, bool MMA, typename Sync, typename Out>
__device__ __forceinline__ void att_unit(const float *q, const T *pk, const T *pv, int P, const float *kb, const float *vb, int L, int d,
                                         int dh, int ch, int n_ch, int gpc, int mma, float *part, int *counter, float *sh, int warp,
                                         int lane, Sync sync, Out out)
{
    if constexpr (MMA && sizeof(T) == 2) {
        if (mma) {
            // chunks 0 .. n_ch - 2: prefix groups on tensor cores; the last chunk: the block's own keys
            const int stride = dh + 2;
            if (ch < n_ch - 1) {
                float *slot = part + (size_t)ch * L * stride;
                if (dh == 128) att_unit_mma<4>(q, pk, pv, P, L, d, ch * gpc, (ch + 1) * gpc, slot, sh, warp, lane, sync);
                else att_unit_mma<2>(q, pk, pv, P, L, d, ch * gpc, (ch + 1) * gpc, slot, sh, warp, lane, sync);
                att_arrive_merge(n_ch, L, dh, part, counter, sh, warp, lane, sync, out);
            } else if (dh == 128) {
                att_unit_per<4>(q, pk, pv, 0, kb, vb, L, d, dh, 0, 1 << 30, ch, n_ch, part, counter, sh, warp, lane, sync, out);
            } else {
                att_unit_per<2>(q, pk, pv, 0, kb, vb, L, d, dh, 0, 1 << 30, ch, n_ch, part, counter, sh, warp, lane, sync, out);
            }
            return;
        }
    }
    // heads of 64 or 128 features, rows 16-byte aligned: the lane's features are consecutive and load as one vector
    if (dh == 128 && (d % 8) == 0)
        att_unit_per<4>(q, pk, pv, P, kb, vb, L, d, dh, ch * gpc, (ch + 1) * gpc, ch, n_ch, part, counter, sh, warp, lane, sync, out);
    else if (dh == 64 && (d % 8) == 0)
        att_unit_per<2>(q, pk, pv, P, kb, vb, L, d, dh, ch * gpc, (ch + 1) * gpc, ch, n_ch, part, counter, sh, warp, lane, sync, out);
    else
        att_unit_per<0>(q, pk, pv, P, kb, vb, L, d, dh, ch * gpc, (ch + 1) * gpc, ch, n_ch, part, counter, sh, warp, lane, sync, out);
}

}  // namespace mrp
