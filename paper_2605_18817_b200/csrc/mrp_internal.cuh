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
    // key / value cache [max_seqs][prefix_cap][d] (context dtype), host copy; lengths per sequence on the device
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
constexpr int kModChainBarInts = 23 * 448 + 1;
cudaError_t sk_module_step(Ctx *c, int n, int L, const int32_t *tokens, const void *hidden0, float *h_state, bool first_step,
                           __nv_bfloat16 *cat16, __nv_bfloat16 *xa, __nv_bfloat16 *xb, __nv_bfloat16 *act16, float *q, float *k,
                           float *v, float *z, int32_t *bar_mem, const int32_t *row_index, int n_masked, int lo_xt, bool f16_lm,
                           float *hidden_out, int32_t *user_status, cudaStream_t st, bool check_only);
// The same for the CUDA-core family (operand rows: fp32 xt).
cudaError_t simt_lm_tail(Ctx *c, const float *logits0, const int32_t *row_index, int M, int K,
                         const mrp_draft_out &out, cudaStream_t st);

// One step of the token-conditioned module (simt_kernels.cu): module forward on CUDA cores, then the
// context's LM-head tail.
cudaError_t module_step(Ctx *c, const int32_t *tokens, const void *hidden0, float *h_state, const float *logits0,
                        const int32_t *row_index, int M, int B, int L, bool first_step, const mrp_draft_out &out,
                        cudaStream_t st);
size_t module_workspace_bytes(const mrp_config &cfg, int n_layers);

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
// One (query position, attention head) by the four warps of a CTA (or of its epilogue warpgroup).  Keys and values:
// the first P rows of the sequence's slab of the prefix cache (type T, written by earlier calls, read through the
// read-only path), then the L rows of the block (fp32, possibly written earlier in this same kernel: read from L2).
// Every warp takes each fourth group of 32 keys: a lane per key for the scores, lanes over the head's features for
// the weighted values, with a running maximum and sum; the four partial results meet in shared memory.
//   sh      kAttShFloats floats of shared memory;  sync(): a barrier over exactly these 128 threads
//   out(c, value) is called once per feature c of the head
// All pointers already point at the head's slice of their row; d is the row stride of all of them.
constexpr int kAttMaxDh = 256;
constexpr int kAttShFloats = kAttMaxDh + 4 * (kAttMaxDh + 2);

__device__ __forceinline__ float att_f(float x) { return x; }
__device__ __forceinline__ float att_f(__nv_bfloat16 x) { return __bfloat162float(x); }

// q_s . row over dh features; vec: rows 16-byte aligned and dh % 8 == 0
__device__ __forceinline__ float att_dot8(const float *q8, const uint4 &u, float s)
{
    const float4 a = *reinterpret_cast<const float4 *>(q8), b = *reinterpret_cast<const float4 *>(q8 + 4);
    const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&u);
    const float2 f0 = __bfloat1622float2(h[0]), f1 = __bfloat1622float2(h[1]), f2 = __bfloat1622float2(h[2]), f3 = __bfloat1622float2(h[3]);
    s = fmaf(a.x, f0.x, s); s = fmaf(a.y, f0.y, s); s = fmaf(a.z, f1.x, s); s = fmaf(a.w, f1.y, s);
    s = fmaf(b.x, f2.x, s); s = fmaf(b.y, f2.y, s); s = fmaf(b.z, f3.x, s); s = fmaf(b.w, f3.y, s);
    return s;
}
__device__ __forceinline__ float att_dot_ro(const float *q_s, const __nv_bfloat16 *row, int dh, bool vec)
{
    float s = 0.f;
    if (vec && (dh & 31) == 0) {
        // 64 bytes of the row per step, the loads of several steps in flight together
        float s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll 4
        for (int c = 0; c < dh; c += 32) {
            const uint4 *r4 = reinterpret_cast<const uint4 *>(row + c);
            const uint4 u0 = __ldg(r4), u1 = __ldg(r4 + 1), u2 = __ldg(r4 + 2), u3 = __ldg(r4 + 3);
            s = att_dot8(q_s + c, u0, s);
            s1 = att_dot8(q_s + c + 8, u1, s1);
            s2 = att_dot8(q_s + c + 16, u2, s2);
            s3 = att_dot8(q_s + c + 24, u3, s3);
        }
        s = (s + s1) + (s2 + s3);
    } else if (vec) {
        for (int c = 0; c < dh; c += 8) s = att_dot8(q_s + c, __ldg(reinterpret_cast<const uint4 *>(row + c)), s);
    } else {
        for (int c = 0; c < dh; ++c) s = fmaf(q_s[c], __bfloat162float(__ldg(row + c)), s);
    }
    return s;
}
__device__ __forceinline__ float att_dot_ro(const float *q_s, const float *row, int dh, bool vec)
{
    float s = 0.f;
    if (vec) {
#pragma unroll 8
        for (int c = 0; c < dh; c += 4) {
            const float4 u = __ldg(reinterpret_cast<const float4 *>(row + c)), a = *reinterpret_cast<const float4 *>(q_s + c);
            s = fmaf(a.x, u.x, s); s = fmaf(a.y, u.y, s); s = fmaf(a.z, u.z, s); s = fmaf(a.w, u.w, s);
        }
    } else {
        for (int c = 0; c < dh; ++c) s = fmaf(q_s[c], __ldg(row + c), s);
    }
    return s;
}
__device__ __forceinline__ float att_dot_cg(const float *q_s, const float *row, int dh, bool vec)
{
    float s = 0.f;
    if (vec) {
        for (int c = 0; c < dh; c += 4) {
            const float4 u = __ldcg(reinterpret_cast<const float4 *>(row + c)), a = *reinterpret_cast<const float4 *>(q_s + c);
            s = fmaf(a.x, u.x, s); s = fmaf(a.y, u.y, s); s = fmaf(a.z, u.z, s); s = fmaf(a.w, u.w, s);
        }
    } else {
        for (int c = 0; c < dh; ++c) s = fmaf(q_s[c], __ldcg(row + c), s);
    }
    return s;
}

template <typename T, typename Sync, typename Out>
__device__ __forceinline__ void att_prefix_item(const float *qi, const T *pk, const T *pv, int P, const float *kb,
                                                const float *vb, int L, int d, int dh, float *sh, int warp, int lane, Sync sync,
                                                Out out)
{
    float *q_s = sh, *part = sh + kAttMaxDh;              // part[w]: maximum, sum, o[dh]
    const int t = warp * 32 + lane;
    for (int c = t; c < dh; c += 128) q_s[c] = __ldcg(qi + c);
    sync();
    const float scale = rsqrtf((float)dh);
    const bool vec = (dh % 8) == 0 && (d % 8) == 0;
    float mx = -INFINITY, sum = 0.f, oacc[kAttMaxDh / 32];
#pragma unroll
    for (int u = 0; u < kAttMaxDh / 32; ++u) oacc[u] = 0.f;
    const int gp = (P + 31) / 32, gb = (L + 31) / 32;
    for (int g = warp; g < gp + gb; g += 4) {
        const bool pre = g < gp;
        const int j0 = pre ? g * 32 : (g - gp) * 32;
        const int left = (pre ? P : L) - j0, cnt = left < 32 ? left : 32;
        float s = -INFINITY;
        if (lane < cnt)
            s = (pre ? att_dot_ro(q_s, pk + (size_t)(j0 + lane) * d, dh, vec) : att_dot_cg(q_s, kb + (size_t)(j0 + lane) * d, dh, vec)) *
                scale;
        float gm = s;
#pragma unroll
        for (int w = 16; w > 0; w >>= 1) gm = fmaxf(gm, __shfl_xor_sync(0xffffffffu, gm, w));
        const float nm = fmaxf(mx, gm), corr = expf(mx - nm);            // (mx = -inf at first: corr = 0)
        const float pj = lane < cnt ? expf(s - nm) : 0.f;
        sum = sum * corr + pj;                                           // per-lane share; corr is the same in every lane
#pragma unroll
        for (int u = 0; u < kAttMaxDh / 32; ++u) oacc[u] *= corr;
        if (pre && cnt == 32) {
            // a full group of prefix rows: the value loads of eight keys in flight together
#pragma unroll 8
            for (int jj = 0; jj < 32; ++jj) {
                const float w = __shfl_sync(0xffffffffu, pj, jj);
                const T *vr = pv + (size_t)(j0 + jj) * d;
#pragma unroll
                for (int u = 0; u < kAttMaxDh / 32; ++u) {
                    const int c = lane + 32 * u;
                    if (c < dh) oacc[u] = fmaf(w, att_f(__ldg(vr + c)), oacc[u]);
                }
            }
        } else {
            for (int jj = 0; jj < cnt; ++jj) {
                const float w = __shfl_sync(0xffffffffu, pj, jj);
                if (pre) {
                    const T *vr = pv + (size_t)(j0 + jj) * d;
#pragma unroll
                    for (int u = 0; u < kAttMaxDh / 32; ++u) {
                        const int c = lane + 32 * u;
                        if (c < dh) oacc[u] = fmaf(w, att_f(__ldg(vr + c)), oacc[u]);
                    }
                } else {
                    const float *vr = vb + (size_t)(j0 + jj) * d;
#pragma unroll
                    for (int u = 0; u < kAttMaxDh / 32; ++u) {
                        const int c = lane + 32 * u;
                        if (c < dh) oacc[u] = fmaf(w, __ldcg(vr + c), oacc[u]);
                    }
                }
            }
        }
        mx = nm;
    }
#pragma unroll
    for (int w = 16; w > 0; w >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, w);
    float *mine = part + warp * (kAttMaxDh + 2);
    if (lane == 0) {
        mine[0] = mx;
        mine[1] = sum;
    }
#pragma unroll
    for (int u = 0; u < kAttMaxDh / 32; ++u) {
        const int c = lane + 32 * u;
        if (c < dh) mine[2 + c] = oacc[u];
    }
    sync();
    // the block has at least one key, so the overall maximum is finite; a warp that had no keys weighs 0
    float top = -INFINITY, e[4], tot = 0.f;
#pragma unroll
    for (int w = 0; w < 4; ++w) top = fmaxf(top, part[w * (kAttMaxDh + 2)]);
#pragma unroll
    for (int w = 0; w < 4; ++w) {
        e[w] = expf(part[w * (kAttMaxDh + 2)] - top);
        tot = fmaf(part[w * (kAttMaxDh + 2) + 1], e[w], tot);
    }
    for (int c = t; c < dh; c += 128) {
        float o = 0.f;
#pragma unroll
        for (int w = 0; w < 4; ++w) o = fmaf(part[w * (kAttMaxDh + 2) + 2 + c], e[w], o);
        out(c, o / tot);
    }
    sync();                                                              // sh is free again
}


}  // namespace mrp
