// C ABI of libmrp_b200.so: argument validation, workspace layout, launch sequencing.
#include <stdlib.h>
#include <string.h>

#include <new>

#include "mrp_internal.cuh"

namespace mrp {

WorkspaceLayout workspace_layout(const mrp_config &cfg)
{
    WorkspaceLayout l;
    memset(&l, 0, sizeof(l));
    const size_t rows = (size_t)cfg.max_rows, d = (size_t)cfg.d, F = (size_t)cfg.d_ff;
    const size_t steps = (size_t)cfg.n_heads + 1;
    size_t off = 0;
    auto take = [&](size_t bytes) { const size_t o = off; off = align_up(off + bytes, 256); return o; };
    l.status = take(64 * sizeof(int32_t));
    l.h0f = take(rows * d * 4);
    l.hcur = take(rows * d * 4);
    // bf16 hi block + lo block each; the few-row kernels put the lo block at a padded row offset
    l.xg = take((rows + 64) * d * 4);
    l.act = take((rows + 64) * F * 4);
    l.xt = take((steps * rows + 32) * d * 4);
    l.sumsq = take((size_t)kSumsqSlices * rows * 4);
    const int v_slices = (cfg.vocab + 31) / 32;      // the narrowest slicing of the CUDA-core LM head
    l.n_slices_max = v_slices < kSimtMaxBlocks ? v_slices : kSimtMaxBlocks;
    if (l.n_slices_max < kSumsqSlices) l.n_slices_max = kSumsqSlices;   // one slice per CTA (tc family)
    l.partials = take((size_t)l.n_slices_max * steps * rows * sizeof(Partial));
    l.dense_row = take((size_t)cfg.max_seqs * (size_t)cfg.block_len * 4);
    l.sk_scratch = take((size_t)kSkScratchBytes);
    l.sk_counters = take((size_t)kSkMaxTiles * 4);
    l.ssq_fix = take((size_t)5 * 128 * 8);
    l.has_f16 = cfg.dtype == MRP_BF16 && !(cfg.flags & (MRP_FLAG_FORCE_SIMT | MRP_FLAG_EXACT_OPERANDS)) &&
                ((long long)cfg.n_heads + 1) * cfg.max_rows >= kF16MinRowSteps && cfg.d % 64 == 0 &&
                cfg.d_ff % 64 == 0 && cfg.vocab % 16 == 0;
    l.w16 = take(l.has_f16 ? (size_t)cfg.vocab * d * 2 : 0);
    l.xt16 = take(l.has_f16 ? (size_t)steps * rows * d * 2 : 0);
    l.kl_partials = take((cfg.flags & MRP_FLAG_TRAINING_KL)
                             ? (size_t)l.n_slices_max * (size_t)cfg.n_heads * rows * sizeof(KlPartial) : 0);
    const bool fp8 = (cfg.flags & MRP_FLAG_FP8_LM) != 0;
    l.w8 = take(fp8 ? (size_t)cfg.vocab * d : 0);
    l.w8_scale = take(fp8 ? (size_t)cfg.vocab * 4 : 0);
    l.xq = take(fp8 ? (size_t)4 * 32 * d : 0);
    l.x8_scale = take(fp8 ? 32 * 4 : 0);
    l.total = off;
    return l;
}

static bool config_ok(const mrp_config *c)
{
    if (!c) return false;
    if (c->d <= 0 || c->d_ff <= 0 || c->vocab <= 0 || c->n_heads < 0 || c->max_rows <= 0 ||
        c->max_seqs <= 0 || c->block_len <= 0 || c->block_len > 1024)
        return false;
    if (c->dtype != MRP_F32 && c->dtype != MRP_BF16) return false;
    if (!(c->rms_eps >= 0.f)) return false;
    if ((long long)c->max_seqs * c->block_len > (1ll << 30)) return false;
    return true;
}

struct DeviceGuard {
    int prev = -1;
    bool switched = false;
    cudaError_t err = cudaSuccess;
    explicit DeviceGuard(int dev)
    {
        err = cudaGetDevice(&prev);
        if (err == cudaSuccess && prev != dev) {
            err = cudaSetDevice(dev);
            switched = (err == cudaSuccess);
        }
    }
    ~DeviceGuard()
    {
        if (switched) cudaSetDevice(prev);
    }
};

}  // namespace mrp

using namespace mrp;

struct mrp_ctx {
    Ctx c;
};

extern "C" {

size_t mrp_workspace_bytes(const mrp_config *cfg)
{
    if (!config_ok(cfg)) return 0;
    return workspace_layout(*cfg).total;
}

int mrp_create(const mrp_config *cfg, const mrp_head_weights *heads, const void *w_lm,
               void *workspace, size_t workspace_bytes, mrp_ctx **out)
{
    if (!out) return MRP_ERR_INVALID_ARG;
    *out = nullptr;
    if (!config_ok(cfg) || !w_lm || !workspace) return MRP_ERR_INVALID_ARG;
    if (cfg->n_heads > 0 && !heads) return MRP_ERR_INVALID_ARG;
    for (int k = 0; k < cfg->n_heads; ++k)
        if (!heads[k].rms_gamma || !heads[k].w_gate || !heads[k].w_up || !heads[k].w_down)
            return MRP_ERR_INVALID_ARG;
    if (((uintptr_t)workspace & 255u) != 0) return MRP_ERR_INVALID_ARG;
    const WorkspaceLayout lay = workspace_layout(*cfg);
    if (workspace_bytes < lay.total) return MRP_ERR_NOMEM;

    DeviceGuard guard(cfg->device);
    if (guard.err != cudaSuccess) return MRP_ERR_CUDA;
    mrp_ctx *ctx = new (std::nothrow) mrp_ctx;
    if (!ctx) return MRP_ERR_NOMEM;
    Ctx &c = ctx->c;
    memset(&c, 0, sizeof(c));
    c.cfg = *cfg;
    c.heads = nullptr;
    if (cfg->n_heads > 0) {
        c.heads = (mrp_head_weights *)malloc(sizeof(mrp_head_weights) * (size_t)cfg->n_heads);
        if (!c.heads) { delete ctx; return MRP_ERR_NOMEM; }
        memcpy(c.heads, heads, sizeof(mrp_head_weights) * (size_t)cfg->n_heads);
    }
    c.w_lm = w_lm;
    c.ws = (char *)workspace;
    c.lay = lay;
    c.launches = 0;
    c.tc_state = nullptr;
    int sm = 0;
    if (cudaDeviceGetAttribute(&sm, cudaDevAttrMultiProcessorCount, cfg->device) != cudaSuccess || sm <= 0) {
        free(c.heads); delete ctx; return MRP_ERR_CUDA;
    }
    c.sm_count = sm;
    c.use_tc = (cfg->dtype == MRP_BF16) && !(cfg->flags & MRP_FLAG_FORCE_SIMT) &&
               tc_supported(*cfg, c.heads, w_lm);
    if ((cfg->flags & MRP_FLAG_REQUIRE_TENSOR_CORES) && !c.use_tc) {
        free(c.heads); delete ctx; return MRP_ERR_UNSUPPORTED;
    }
    if ((cfg->flags & MRP_FLAG_FP8_LM) && (!c.use_tc || !fp8_lm_supported(*cfg))) {
        free(c.heads); delete ctx; return MRP_ERR_UNSUPPORTED;
    }
    {
        const long long dense = (long long)cfg->max_seqs * cfg->block_len;
        c.input_rows = (int)(dense > cfg->max_rows ? dense : cfg->max_rows);
    }
    if (c.use_tc) {
        if (tc_create(&c) != cudaSuccess) { free(c.heads); delete ctx; return MRP_ERR_CUDA; }
        if ((cfg->flags & MRP_FLAG_FP8_LM) && fp8_lm_create(&c) != cudaSuccess) {
            tc_destroy(&c); free(c.heads); delete ctx; return MRP_ERR_CUDA;
        }
    }
    if (cudaMemset(c.ws + lay.status, 0, 64 * sizeof(int32_t)) != cudaSuccess) {
        if (c.use_tc) tc_destroy(&c);
        free(c.heads); delete ctx; return MRP_ERR_CUDA;
    }
    *out = ctx;
    return MRP_OK;
}

static void prof_release(Ctx &c)
{
    if (c.prof_events) {
        for (int i = 0; i < kProfSlots * kProfMarks; ++i)
            if (c.prof_events[i]) cudaEventDestroy(c.prof_events[i]);
        free(c.prof_events);
        c.prof_events = nullptr;
    }
    c.prof_enabled = false;
    c.prof_calls = 0;
}

int mrp_profile_enable(mrp_ctx *ctx, int32_t enable)
{
    if (!ctx) return MRP_ERR_INVALID_ARG;
    Ctx &c = ctx->c;
    DeviceGuard guard(c.cfg.device);
    if (guard.err != cudaSuccess) return MRP_ERR_CUDA;
    if (!enable) { prof_release(c); return MRP_OK; }
    if (!c.prof_events) {
        c.prof_events = (cudaEvent_t *)calloc((size_t)kProfSlots * kProfMarks, sizeof(cudaEvent_t));
        if (!c.prof_events) return MRP_ERR_NOMEM;
        for (int i = 0; i < kProfSlots * kProfMarks; ++i)
            if (cudaEventCreate(&c.prof_events[i]) != cudaSuccess) { prof_release(c); return MRP_ERR_CUDA; }
    }
    c.prof_calls = 0;
    c.prof_enabled = true;
    return MRP_OK;
}

int mrp_profile_read(mrp_ctx *ctx, float *ms_phase, int32_t *n_calls)
{
    if (!ctx || !ms_phase || !n_calls) return MRP_ERR_INVALID_ARG;
    Ctx &c = ctx->c;
    ms_phase[0] = ms_phase[1] = ms_phase[2] = 0.f;
    *n_calls = 0;
    if (!c.prof_enabled) return MRP_OK;
    DeviceGuard guard(c.cfg.device);
    if (guard.err != cudaSuccess) return MRP_ERR_CUDA;
    const int n = (int)(c.prof_calls < kProfSlots ? c.prof_calls : kProfSlots);
    double acc[3] = {0, 0, 0};
    for (int i = 0; i < n; ++i) {
        cudaEvent_t *ev = c.prof_events + (size_t)i * kProfMarks;
        for (int ph = 0; ph < 3; ++ph) {
            float ms = 0.f;
            if (cudaEventElapsedTime(&ms, ev[ph], ev[ph + 1]) != cudaSuccess) return MRP_ERR_CUDA;
            acc[ph] += ms;
        }
    }
    for (int ph = 0; ph < 3; ++ph) ms_phase[ph] = (float)acc[ph];
    *n_calls = n;
    c.prof_calls = 0;
    return MRP_OK;
}

void mrp_destroy(mrp_ctx *ctx)
{
    if (!ctx) return;
    prof_release(ctx->c);
    if (ctx->c.use_tc) tc_destroy(&ctx->c);
    free(ctx->c.module_layers);
    free(ctx->c.prefix_layers);
    free(ctx->c.heads);
    delete ctx;
}

static int draft_call(mrp_ctx *ctx, const void *hidden, const float *logits0, bool from_hidden,
                      const void *final_gamma, const int32_t *row_index, int32_t M, int32_t K,
                      const mrp_draft_out *out, void *cuda_stream, const float *teacher = nullptr,
                      float *kl = nullptr, bool l0_bf16 = false)
{
    if (!ctx || !out) return MRP_ERR_INVALID_ARG;
    Ctx &c = ctx->c;
    c.teacher = teacher;
    c.kl_out = kl;
    c.l0_bf16 = l0_bf16;
    if (M < 0 || M > c.cfg.max_rows || K < 0 || K > c.cfg.n_heads) return MRP_ERR_INVALID_ARG;
    c.launches = 0;
    if (M == 0) return MRP_OK;
    if (c.use_fp8_lm && (K < 1 || teacher)) return MRP_ERR_UNSUPPORTED;   // the 8-bit LM head serves drafting passes with K >= 1
    if (!hidden || (!from_hidden && !logits0) || !out->conf || !out->lse || !out->token) return MRP_ERR_INVALID_ARG;
    if (!row_index && M > c.input_rows) return MRP_ERR_INVALID_ARG;      // rows 0..M-1 must exist
    if (((uintptr_t)hidden & 15u) || ((uintptr_t)logits0 & 15u)) return MRP_ERR_INVALID_ARG;
    DeviceGuard guard(c.cfg.device);
    if (guard.err != cudaSuccess) return MRP_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    c.err[0] = 0;
    c.from_hidden = from_hidden;
    c.final_gamma = from_hidden ? final_gamma : nullptr;
    cudaError_t e = c.use_tc ? tc_draft(&c, hidden, logits0, row_index, M, K, *out, st)
                             : simt_draft(&c, hidden, logits0, row_index, M, K, *out, st);
    if (e != cudaSuccess && !c.err[0]) note_err(&c, e, "mrp_draft");
    return e == cudaSuccess ? MRP_OK : MRP_ERR_CUDA;
}

int mrp_draft(mrp_ctx *ctx, const void *hidden, const float *logits0, const int32_t *row_index,
              int32_t M, int32_t K, const mrp_draft_out *out, void *cuda_stream)
{
    return draft_call(ctx, hidden, logits0, false, nullptr, row_index, M, K, out, cuda_stream);
}

int mrp_draft_bf16_logits(mrp_ctx *ctx, const void *hidden, const void *logits0_bf16, const int32_t *row_index,
                          int32_t M, int32_t K, const mrp_draft_out *out, void *cuda_stream)
{
    return draft_call(ctx, hidden, (const float *)logits0_bf16, false, nullptr, row_index, M, K, out, cuda_stream,
                      nullptr, nullptr, true);
}

int mrp_draft_kl(mrp_ctx *ctx, const void *hidden, const float *logits0, const float *teacher,
                 const int32_t *row_index, int32_t M, int32_t K, const mrp_draft_out *out, float *kl,
                 void *cuda_stream)
{
    if (!ctx) return MRP_ERR_INVALID_ARG;
    if (!(ctx->c.cfg.flags & MRP_FLAG_TRAINING_KL)) return MRP_ERR_UNSUPPORTED;
    if (K < 1 || (M > 0 && (!teacher || !kl)) || ((uintptr_t)teacher & 15u)) return MRP_ERR_INVALID_ARG;
    return draft_call(ctx, hidden, logits0, false, nullptr, row_index, M, K, out, cuda_stream, teacher, kl);
}

int mrp_draft_from_hidden(mrp_ctx *ctx, const void *hidden, const void *final_norm_gamma,
                          const int32_t *row_index, int32_t M, int32_t K, const mrp_draft_out *out,
                          void *cuda_stream)
{
    return draft_call(ctx, hidden, nullptr, true, final_norm_gamma, row_index, M, K, out, cuda_stream);
}

int mrp_reveal_remask(mrp_ctx *ctx, const float *conf, const int32_t *token,
                      const int32_t *row_index, int32_t M, int32_t K, int32_t B, int32_t L,
                      const mrp_select_params *params, const mrp_select_out *out, void *cuda_stream)
{
    if (!ctx || !params || !out) return MRP_ERR_INVALID_ARG;
    Ctx &c = ctx->c;
    if (B < 1 || B > c.cfg.max_seqs || L < 1 || L > c.cfg.block_len) return MRP_ERR_INVALID_ARG;
    if (M < 0 || (long long)M > (long long)B * L || K < 0) return MRP_ERR_INVALID_ARG;
    if (M > 0 && (!conf || !token)) return MRP_ERR_INVALID_ARG;
    if (params->mode != MRP_SELECT_STATIC && params->mode != MRP_SELECT_DYNAMIC_REMASK)
        return MRP_ERR_INVALID_ARG;
    if (params->r_reveal < 0 || params->r_draft < 0) return MRP_ERR_INVALID_ARG;
    if (params->remask_policy < 0 || params->remask_policy > 3) return MRP_ERR_INVALID_ARG;
    if (params->mode == MRP_SELECT_DYNAMIC_REMASK && params->remask_policy == 2 && M > 0 && !params->conf_first)
        return MRP_ERR_INVALID_ARG;
    if (!out->reveal_mask || !out->remask_mask || !out->out_token || !out->step_of || !out->draft_len)
        return MRP_ERR_INVALID_ARG;
    const int Kd = K * params->r_draft;
    if (Kd > 0 && (!out->draft_pos || !out->draft_tok)) return MRP_ERR_INVALID_ARG;
    c.launches = 0;
    DeviceGuard guard(c.cfg.device);
    if (guard.err != cudaSuccess) return MRP_ERR_CUDA;
    cudaError_t e = launch_select(&c, conf, token, row_index, M, K, B, L, *params, *out,
                                  (cudaStream_t)cuda_stream);
    return e == cudaSuccess ? MRP_OK : MRP_ERR_CUDA;
}

int mrp_verify(mrp_ctx *ctx, const int32_t *draft_tok, const int32_t *verify_tok,
               const int32_t *draft_len, int32_t B, int32_t Kd, int32_t positionwise,
               int32_t *accept_len, int8_t *accept_mask, void *cuda_stream)
{
    if (!ctx) return MRP_ERR_INVALID_ARG;
    Ctx &c = ctx->c;
    if (B < 0 || B > c.cfg.max_seqs || Kd < 0) return MRP_ERR_INVALID_ARG;
    c.launches = 0;
    if (B == 0) return MRP_OK;
    if (!draft_len || !accept_len) return MRP_ERR_INVALID_ARG;
    if (Kd > 0 && (!draft_tok || !verify_tok || !accept_mask)) return MRP_ERR_INVALID_ARG;
    DeviceGuard guard(c.cfg.device);
    if (guard.err != cudaSuccess) return MRP_ERR_CUDA;
    cudaError_t e = launch_verify(&c, draft_tok, verify_tok, draft_len, B, Kd, positionwise ? 1 : 0,
                                  accept_len, accept_mask, (cudaStream_t)cuda_stream);
    return e == cudaSuccess ? MRP_OK : MRP_ERR_CUDA;
}

static bool module_ok(const mrp_config *cfg, const mrp_module_weights *w)
{
    if (!cfg || !w || w->n_layers < 0 || w->n_layers > 64 || w->n_attn_heads < 1 || cfg->d % w->n_attn_heads) return false;
    if (w->emb_rows < 1 || w->mask_token < 0 || w->mask_token >= w->emb_rows || !w->emb || !w->w_proj) return false;
    if (w->n_layers > 0 && !w->layers) return false;
    for (int l = 0; l < w->n_layers; ++l) {
        const mrp_module_layer &y = w->layers[l];
        if (!y.g_attn || !y.w_q || !y.w_k || !y.w_v || !y.w_o || !y.g_mlp || !y.w_gate || !y.w_up || !y.w_down) return false;
    }
    return true;
}

size_t mrp_module_workspace_bytes(const mrp_config *cfg, const mrp_module_weights *w)
{
    if (!config_ok(cfg) || !module_ok(cfg, w)) return 0;
    return module_workspace_bytes(*cfg, w->n_layers);
}

int mrp_module_attach(mrp_ctx *ctx, const mrp_module_weights *w, void *workspace, size_t workspace_bytes)
{
    if (!ctx || !workspace || ((uintptr_t)workspace & 255u)) return MRP_ERR_INVALID_ARG;
    Ctx &c = ctx->c;
    if (!module_ok(&c.cfg, w)) return MRP_ERR_INVALID_ARG;
    if (workspace_bytes < module_workspace_bytes(c.cfg, w->n_layers)) return MRP_ERR_NOMEM;
    mrp_module_layer *copy = nullptr;
    if (w->n_layers > 0) {
        copy = (mrp_module_layer *)malloc(sizeof(mrp_module_layer) * (size_t)w->n_layers);
        if (!copy) return MRP_ERR_NOMEM;
        memcpy(copy, w->layers, sizeof(mrp_module_layer) * (size_t)w->n_layers);
    }
    free(c.module_layers);
    c.module_layers = copy;
    c.module = *w;
    c.module.layers = copy;
    c.module_ws = (char *)workspace;
    c.has_module = true;
    free(c.prefix_layers);                     // a prefix belongs to the module it was attached for
    c.prefix_layers = nullptr;
    c.has_prefix = false;
    return MRP_OK;
}

int mrp_module_set_prefix(mrp_ctx *ctx, const mrp_module_kv *layers, const int32_t *prefix_len, int32_t prefix_cap,
                          int32_t append)
{
    if (!ctx) return MRP_ERR_INVALID_ARG;
    Ctx &c = ctx->c;
    if (!c.has_module) return MRP_ERR_UNSUPPORTED;
    if (!layers) {
        free(c.prefix_layers);
        c.prefix_layers = nullptr;
        c.has_prefix = false;
        return MRP_OK;
    }
    const int D = c.module.n_layers;
    if (!prefix_len || prefix_cap < 0 || (long long)prefix_cap + c.cfg.block_len > 0x7fffffffLL / 2) return MRP_ERR_INVALID_ARG;
    for (int l = 0; l < D; ++l)
        if (!layers[l].k || !layers[l].v || ((uintptr_t)layers[l].k & 15u) || ((uintptr_t)layers[l].v & 15u))
            return MRP_ERR_INVALID_ARG;
    if (c.cfg.d / c.module.n_attn_heads > kAttMaxDh) return MRP_ERR_UNSUPPORTED;
    mrp_module_kv *copy = (mrp_module_kv *)malloc(sizeof(mrp_module_kv) * (size_t)(D > 0 ? D : 1));
    if (!copy) return MRP_ERR_NOMEM;
    if (D > 0) memcpy(copy, layers, sizeof(mrp_module_kv) * (size_t)D);
    free(c.prefix_layers);
    c.prefix_layers = copy;
    c.prefix_len = prefix_len;
    c.prefix_cap = prefix_cap;
    c.prefix_append = append != 0;
    c.has_prefix = true;
    return MRP_OK;
}

static int module_call(mrp_ctx *ctx, const int32_t *tokens, const void *hidden0, float *h_state, const float *logits0,
                       const int32_t *row_index, int32_t M, int32_t B, int32_t L, int32_t first_step,
                       const mrp_draft_out *out, void *cuda_stream, const float *teacher, float *kl)
{
    if (!ctx || !out) return MRP_ERR_INVALID_ARG;
    Ctx &c = ctx->c;
    if (!c.has_module) return MRP_ERR_UNSUPPORTED;
    if (B < 1 || B > c.cfg.max_seqs || L < 1 || L > c.cfg.block_len) return MRP_ERR_INVALID_ARG;
    if (M < 0 || M > c.cfg.max_rows || (long long)M > (long long)B * L) return MRP_ERR_INVALID_ARG;
    if (!tokens || !hidden0 || !h_state || ((uintptr_t)hidden0 & 15u) || ((uintptr_t)h_state & 15u)) return MRP_ERR_INVALID_ARG;
    if (M > 0 && (!logits0 || ((uintptr_t)logits0 & 15u) || !out->conf || !out->lse || !out->token)) return MRP_ERR_INVALID_ARG;
    c.launches = 0;
    DeviceGuard guard(c.cfg.device);
    if (guard.err != cudaSuccess) return MRP_ERR_CUDA;
    c.err[0] = 0;
    c.from_hidden = false; c.final_gamma = nullptr; c.l0_bf16 = false;
    c.teacher = M > 0 ? teacher : nullptr; c.kl_out = M > 0 ? kl : nullptr;
    const int saved_rows = c.input_rows;
    c.input_rows = B * L;                       // the dense arrays of this call have B * L rows
    cudaError_t e = module_step(&c, tokens, hidden0, h_state, logits0, row_index, M, B, L, first_step != 0, *out,
                                (cudaStream_t)cuda_stream);
    c.input_rows = saved_rows;
    c.teacher = nullptr; c.kl_out = nullptr;
    if (e != cudaSuccess && !c.err[0]) note_err(&c, e, "mrp_module_step");
    return e == cudaSuccess ? MRP_OK : MRP_ERR_CUDA;
}

int mrp_module_step(mrp_ctx *ctx, const int32_t *tokens, const void *hidden0, float *h_state, const float *logits0,
                    const int32_t *row_index, int32_t M, int32_t B, int32_t L, int32_t first_step,
                    const mrp_draft_out *out, void *cuda_stream)
{
    return module_call(ctx, tokens, hidden0, h_state, logits0, row_index, M, B, L, first_step, out, cuda_stream, nullptr, nullptr);
}

int mrp_module_step_kl(mrp_ctx *ctx, const int32_t *tokens, const void *hidden0, float *h_state, const float *logits0,
                       const float *teacher, const int32_t *row_index, int32_t M, int32_t B, int32_t L, int32_t first_step,
                       const mrp_draft_out *out, float *kl, void *cuda_stream)
{
    if (!ctx) return MRP_ERR_INVALID_ARG;
    if (!(ctx->c.cfg.flags & MRP_FLAG_TRAINING_KL) || ctx->c.use_fp8_lm) return MRP_ERR_UNSUPPORTED;
    if ((M > 0 && (!teacher || !kl)) || ((uintptr_t)teacher & 15u)) return MRP_ERR_INVALID_ARG;
    return module_call(ctx, tokens, hidden0, h_state, logits0, row_index, M, B, L, first_step, out, cuda_stream, teacher, kl);
}

int mrp_quantised_lm_head(mrp_ctx *ctx, const uint8_t **codes, const float **scales)
{
    if (!ctx || !codes || !scales) return MRP_ERR_INVALID_ARG;
    if (!ctx->c.use_fp8_lm) return MRP_ERR_UNSUPPORTED;
    *codes = (const uint8_t *)(ctx->c.ws + ctx->c.lay.w8);
    *scales = (const float *)(ctx->c.ws + ctx->c.lay.w8_scale);
    return MRP_OK;
}

int mrp_set_input_rows(mrp_ctx *ctx, int32_t n_rows)
{
    if (!ctx) return MRP_ERR_INVALID_ARG;
    const mrp_config &cfg = ctx->c.cfg;
    const long long dense = (long long)cfg.max_seqs * cfg.block_len;
    const long long most = dense > cfg.max_rows ? dense : (long long)cfg.max_rows;
    if (n_rows < 1 || n_rows > most) return MRP_ERR_INVALID_ARG;
    ctx->c.input_rows = n_rows;
    return MRP_OK;
}

int mrp_fetch_status(mrp_ctx *ctx, int32_t *dst, int32_t clear, void *cuda_stream)
{
    if (!ctx || !dst) return MRP_ERR_INVALID_ARG;
    Ctx &c = ctx->c;
    DeviceGuard guard(c.cfg.device);
    if (guard.err != cudaSuccess) return MRP_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    int32_t *word = (int32_t *)(c.ws + c.lay.status);
    if (cudaMemcpyAsync(dst, word, sizeof(int32_t), cudaMemcpyDeviceToDevice, st) != cudaSuccess) return MRP_ERR_CUDA;
    if (clear && cudaMemsetAsync(word, 0, sizeof(int32_t), st) != cudaSuccess) return MRP_ERR_CUDA;
    return MRP_OK;
}

int mrp_set_logits0_event(mrp_ctx *ctx, void *cuda_event)
{
    if (!ctx) return MRP_ERR_INVALID_ARG;
    ctx->c.l0_event = (cudaEvent_t)cuda_event;
    return MRP_OK;
}

int mrp_commit(mrp_ctx *ctx, const mrp_select_out *sel, const int8_t *accept_mask, int32_t B, int32_t L,
               int32_t Kd, const mrp_block_state *state, void *cuda_stream)
{
    if (!ctx || !sel || !state) return MRP_ERR_INVALID_ARG;
    Ctx &c = ctx->c;
    if (B < 1 || B > c.cfg.max_seqs || L < 1 || L > c.cfg.block_len || Kd < 0) return MRP_ERR_INVALID_ARG;
    if (!state->tokens || !state->row_index || !state->n_masked || !state->block_masked) return MRP_ERR_INVALID_ARG;
    if (!sel->out_token || (accept_mask && !sel->step_of)) return MRP_ERR_INVALID_ARG;
    if (accept_mask && Kd > 0 && (!sel->draft_pos || !sel->draft_tok)) return MRP_ERR_INVALID_ARG;
    c.launches = 0;
    DeviceGuard guard(c.cfg.device);
    if (guard.err != cudaSuccess) return MRP_ERR_CUDA;
    c.err[0] = 0;
    cudaError_t e = launch_commit(&c, *sel, accept_mask, B, L, Kd, *state, (cudaStream_t)cuda_stream);
    return e == cudaSuccess ? MRP_OK : MRP_ERR_CUDA;
}

int mrp_selftest_wait_timeout(mrp_ctx *ctx, int32_t *status, void *cuda_stream)
{
    if (!ctx) return MRP_ERR_INVALID_ARG;
    Ctx &c = ctx->c;
    DeviceGuard guard(c.cfg.device);
    if (guard.err != cudaSuccess) return MRP_ERR_CUDA;
    return tc_selftest_timeout(&c, status, (cudaStream_t)cuda_stream) == cudaSuccess ? MRP_OK : MRP_ERR_CUDA;
}

int32_t mrp_last_launch_count(const mrp_ctx *ctx) { return ctx ? ctx->c.launches : 0; }

const char *mrp_last_error(const mrp_ctx *ctx) { return ctx ? ctx->c.err : ""; }

const char *mrp_kernel_family(const mrp_ctx *ctx)
{
    if (!ctx) return "none";
    return ctx->c.use_tc ? "tcgen05" : "simt";
}

const char *mrp_status_string(int status)
{
    switch (status) {
    case MRP_OK: return "ok";
    case MRP_ERR_INVALID_ARG: return "invalid argument";
    case MRP_ERR_UNSUPPORTED: return "unsupported shape";
    case MRP_ERR_CUDA: return "CUDA error";
    case MRP_ERR_NOMEM: return "workspace too small or out of host memory";
    case MRP_ERR_NONFINITE: return "non-finite values";
    case MRP_ERR_TIMEOUT: return "device wait timed out";
    case MRP_ERR_CAPACITY: return "size exceeds the fixed built-in scratch capacity";
    default: return "unknown status";
    }
}

}  // extern "C"
