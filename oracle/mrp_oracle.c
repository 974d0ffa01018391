/*
 * MRP drafting step -- CPU oracle (TEST INFRASTRUCTURE, not a product path).
 *
 * A plain, slow, fp64 restatement of what one Multi-token Residual Prediction
 * drafting step computes, written from the paper's definitions:
 *   - confidence = top-1 softmax probability of a position (Sec. 2, "Denoising Loop");
 *   - the chain  Delta,delta <- g(x_t,h);  h <- h+Delta;  l <- l+delta  repeated K times
 *     (Algorithm 2, inner loop; Algorithm 3, "MRP drafting"; Algorithm 4, "MRP forward");
 *   - delta is produced by the backbone's own LM head applied to the module output (Sec. 3.2);
 *   - static reveal = the r most confident still-masked positions of the block,
 *     dynamic reveal = every masked position whose confidence clears tau, at least one
 *     per step (Sec. 4.1, "Denoising Mode");
 *   - remask = revoke positions of the reveal set whose updated confidence is below the
 *     same tau (Algorithm 4; Sec. 3.4 "Remasking decoding");
 *   - max-accept cap m = min(max(floor(0.7 n), 5), L) (Sec. 4.4);
 *   - verification = a drafted token is accepted iff it equals the backbone's argmax
 *     (Algorithm 3), with the prefix semantics of Figure 1(d).
 * The head g is the reduced module of the benchmark configurations: RMSNorm followed by a
 * SwiGLU MLP (no biases), whose output r is both the hidden residual Delta and the
 * vector sent through the LM head (delta = W_lm r).
 *
 * Only tests, the smoke check and the benchmark's cpu_baseline leg may call this file.
 * It shares no code, header, table or constant with the CUDA path.  Inputs are float32
 * arrays holding exactly the values the GPU sees (bf16 values are exact in float32);
 * every arithmetic step is done in double.  There is no blocking, fusion or reordering
 * beyond the loops written here; OpenMP only spreads independent output elements over
 * cores.
 *
 * Parity pins live in tests/ (zero-residual heads, softmax normalisation, linearity of the
 * chain in the residual, brute force on tiny vocabularies, a second implementation on
 * library routines, closed forms for the cap and the accepted-prefix length; for the base
 * logits computed from the hidden states: exact agreement with the precomputed-logits pass on
 * integer data, l_k = W_lm h_k without a final norm, the one-hot closed form and the scale
 * invariance of the final norm).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int mrp_oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Softmax statistics of one logit row (Sec. 2): maximum, lowest-index argmax,
 * log-sum-exp, confidence = exp(max - lse), and the gap between the two largest logits. */
static void softmax_stats(const double *l, int V, double *conf, double *lse, int32_t *tok,
                          double *margin)
{
    double mx = l[0];
    int32_t arg = 0;
    for (int v = 1; v < V; ++v)
        if (l[v] > mx) { mx = l[v]; arg = v; }
    double second = -INFINITY;
    for (int v = 0; v < V; ++v)
        if (v != arg && l[v] > second) second = l[v];
    double S = 0.0;
    for (int v = 0; v < V; ++v) S += exp(l[v] - mx);
    double L = mx + log(S);
    *conf = exp(mx - L);
    *lse = L;
    *tok = arg;
    *margin = (V > 1) ? (mx - second) : INFINITY;
}

/* Forward KL divergence KL(softmax(t) || softmax(l)) of two logit rows (Eq. (3)), from the
 * definition: sum_v p_v (log p_v - log q_v) with p = softmax(t), q = softmax(l). */
static double kl_rows(const double *t, const double *l, int V)
{
    double mt = t[0], ml = l[0];
    for (int v = 1; v < V; ++v) { if (t[v] > mt) mt = t[v]; if (l[v] > ml) ml = l[v]; }
    double st = 0.0, sl = 0.0;
    for (int v = 0; v < V; ++v) { st += exp(t[v] - mt); sl += exp(l[v] - ml); }
    const double lse_t = mt + log(st), lse_l = ml + log(sl);
    double kl = 0.0;
    for (int v = 0; v < V; ++v) {
        const double logp = t[v] - lse_t, logq = l[v] - lse_l;
        kl += exp(logp) * (logp - logq);
    }
    return kl;
}

/*
 * One drafting pass over M masked rows (Algorithm 2, lines "for k = 1..K").
 *   hidden  [n_rows, d]   backbone hidden states h
 *   logits0 [n_rows, V]   backbone logits l
 *   row_index [M] or NULL rows of the dense arrays that are masked (NULL = 0..M-1)
 *   gamma/w_gate/w_up/w_down: K pointers each, head k (1-based) = entry k-1;
 *       gamma [d], w_gate [F,d], w_up [F,d], w_down [d,F], row-major [out,in]
 *   w_lm [V, d]
 * Outputs, step-major, k = 0 is the backbone's own logits:
 *   conf, lse, margin [(K+1), M] double; token [(K+1), M] int32
 *   logits_out  optional [K, M, V]  (l after step k = 1..K)
 *   hidden_out  optional [M, d]     (h after step K)
 *   conf_first  optional [(K+1), M] softmax probability, under step k's logits, of the row's
 *               step-0 argmax token (the token a reveal at step 0 commits; Algorithm 4 remasks by
 *               the confidence of the updated logits, and this is the variant that follows the
 *               committed token itself)
 * Returns 0, or -1 on allocation failure / bad arguments.
 */
static int draft_rows(int d, int F, int V, int K, int M, double eps,
                      const float *hidden, const float *logits0, int from_hidden,
                      const float *final_gamma, const int32_t *row_index,
                      const float *const *gamma, const float *const *w_gate,
                      const float *const *w_up, const float *const *w_down,
                      const float *w_lm,
                      double *conf, double *lse, int32_t *token, double *margin,
                      double *logits_out, double *hidden_out, double *conf_first,
                      const float *teacher, double *kl)
{
    if (d <= 0 || F <= 0 || V <= 0 || K < 0 || M < 0) return -1;
    if ((teacher != NULL) != (kl != NULL)) return -1;
    double *h = (double *)malloc(sizeof(double) * (size_t)d);
    double *xh = (double *)malloc(sizeof(double) * (size_t)d);
    double *a = (double *)malloc(sizeof(double) * (size_t)F);
    double *r = (double *)malloc(sizeof(double) * (size_t)d);
    double *l = (double *)malloc(sizeof(double) * (size_t)V);
    double *tt = (double *)malloc(sizeof(double) * (size_t)V);
    if (!h || !xh || !a || !r || !l || !tt) { free(h); free(xh); free(a); free(r); free(l); free(tt); return -1; }

    for (int m = 0; m < M; ++m) {
        const size_t row = row_index ? (size_t)row_index[m] : (size_t)m;
        for (int j = 0; j < d; ++j) h[j] = (double)hidden[row * (size_t)d + j];
        if (!from_hidden) {
            for (int v = 0; v < V; ++v) l[v] = (double)logits0[row * (size_t)V + v];
        } else {
            /* l = W_lm n, n = h (final_gamma NULL) or RMSNorm(h) * final_gamma: the backbone's
             * own LM head applied to the same hidden states ("h, l <- f(x_t)") */
            double rstd0 = 1.0;
            if (final_gamma) {
                double ss0 = 0.0;
                for (int j = 0; j < d; ++j) ss0 += h[j] * h[j];
                rstd0 = 1.0 / sqrt(ss0 / (double)d + eps);
            }
            for (int j = 0; j < d; ++j) xh[j] = final_gamma ? h[j] * rstd0 * (double)final_gamma[j] : h[j];
#pragma omp parallel for schedule(static)
            for (int v = 0; v < V; ++v) {
                double s = 0.0;
                const float *wr = w_lm + (size_t)v * d;
                for (int j = 0; j < d; ++j) s += (double)wr[j] * xh[j];
                l[v] = s;
            }
        }
        softmax_stats(l, V, &conf[m], &lse[m], &token[m], &margin[m]);
        if (conf_first) conf_first[m] = conf[m];

        for (int k = 1; k <= K; ++k) {
            const float *g_k = gamma[k - 1];
            const float *wg = w_gate[k - 1], *wu = w_up[k - 1], *wd = w_down[k - 1];
            /* RMSNorm: xh = h / sqrt(mean(h^2) + eps) * gamma */
            double ss = 0.0;
            for (int j = 0; j < d; ++j) ss += h[j] * h[j];
            const double rstd = 1.0 / sqrt(ss / (double)d + eps);
            for (int j = 0; j < d; ++j) xh[j] = h[j] * rstd * (double)g_k[j];
            /* SwiGLU: a = silu(W_g xh) * (W_u xh), silu(x) = x / (1 + exp(-x)) */
#pragma omp parallel for schedule(static)
            for (int f = 0; f < F; ++f) {
                double g = 0.0, u = 0.0;
                const float *wgr = wg + (size_t)f * d, *wur = wu + (size_t)f * d;
                for (int j = 0; j < d; ++j) g += (double)wgr[j] * xh[j];
                for (int j = 0; j < d; ++j) u += (double)wur[j] * xh[j];
                a[f] = g / (1.0 + exp(-g)) * u;
            }
            /* r = W_d a : the hidden residual Delta */
#pragma omp parallel for schedule(static)
            for (int j = 0; j < d; ++j) {
                double s = 0.0;
                const float *wdr = wd + (size_t)j * F;
                for (int f = 0; f < F; ++f) s += (double)wdr[f] * a[f];
                r[j] = s;
            }
            /* h <- h + Delta */
            for (int j = 0; j < d; ++j) h[j] += r[j];
            /* l <- l + delta, delta = W_lm Delta (shared LM head) */
#pragma omp parallel for schedule(static)
            for (int v = 0; v < V; ++v) {
                double s = 0.0;
                const float *wr = w_lm + (size_t)v * d;
                for (int j = 0; j < d; ++j) s += (double)wr[j] * r[j];
                l[v] += s;
            }
            const size_t o = (size_t)k * M + m;
            softmax_stats(l, V, &conf[o], &lse[o], &token[o], &margin[o]);
            /* probability, under the updated logits, of the token that was on top at step 0 */
            if (conf_first) conf_first[o] = exp(l[token[m]] - lse[o]);
            /* training objective of this unrolled step (Eq. (3), Algorithm 1): the teacher logits of the
             * step against the corrected logits l = l_t + delta */
            if (teacher) {
                const float *tr = teacher + ((size_t)(k - 1) * M + m) * (size_t)V;
                for (int v = 0; v < V; ++v) tt[v] = (double)tr[v];
                kl[(size_t)(k - 1) * M + m] = kl_rows(tt, l, V);
            }
            if (logits_out)
                memcpy(logits_out + ((size_t)(k - 1) * M + m) * V, l, sizeof(double) * (size_t)V);
        }
        if (hidden_out) memcpy(hidden_out + (size_t)m * d, h, sizeof(double) * (size_t)d);
    }
    free(h); free(xh); free(a); free(r); free(l); free(tt);
    return 0;
}

int mrp_oracle_draft(int d, int F, int V, int K, int M, double eps,
                     const float *hidden, const float *logits0, const int32_t *row_index,
                     const float *const *gamma, const float *const *w_gate,
                     const float *const *w_up, const float *const *w_down,
                     const float *w_lm,
                     double *conf, double *lse, int32_t *token, double *margin,
                     double *logits_out, double *hidden_out, double *conf_first)
{
    if (!logits0) return -1;
    return draft_rows(d, F, V, K, M, eps, hidden, logits0, 0, NULL, row_index, gamma, w_gate, w_up, w_down,
                      w_lm, conf, lse, token, margin, logits_out, hidden_out, conf_first, NULL, NULL);
}

/*
 * The drafting pass with the training objective (Algorithm 1; Eq. (3)): teacher [K, M, V] holds, for
 * every unrolled step k = 1..K and masked row m, the backbone's logits on the sequence that has the
 * step's ground-truth tokens revealed (l_{t-1} in the paper's one-step notation); kl [K, M] receives
 * KL(softmax(teacher_k) || softmax(l_k)), l_k = l_{k-1} + delta_k the corrected logits of the step.
 */
int mrp_oracle_draft_kl(int d, int F, int V, int K, int M, double eps,
                        const float *hidden, const float *logits0, const int32_t *row_index,
                        const float *const *gamma, const float *const *w_gate,
                        const float *const *w_up, const float *const *w_down,
                        const float *w_lm, const float *teacher,
                        double *conf, double *lse, int32_t *token, double *margin, double *kl)
{
    if (!logits0 || !teacher || !kl) return -1;
    return draft_rows(d, F, V, K, M, eps, hidden, logits0, 0, NULL, row_index, gamma, w_gate, w_up, w_down,
                      w_lm, conf, lse, token, margin, NULL, NULL, NULL, teacher, kl);
}

/*
 * The same pass when the backbone hands over hidden states only (Algorithm 2: h and l come out
 * of one forward, and Sec. 3.2: the module reuses the backbone's LM head): l_0 = W_lm n_0 with
 * n_0 = h_0, or n_0 = RMSNorm(h_0) * final_gamma when the hidden states are taken before the
 * backbone's final norm (final_gamma [d], NULL = none).  Everything else as mrp_oracle_draft.
 */
int mrp_oracle_draft_from_hidden(int d, int F, int V, int K, int M, double eps,
                                 const float *hidden, const float *final_gamma, const int32_t *row_index,
                                 const float *const *gamma, const float *const *w_gate,
                                 const float *const *w_up, const float *const *w_down,
                                 const float *w_lm,
                                 double *conf, double *lse, int32_t *token, double *margin,
                                 double *logits_out, double *hidden_out, double *conf_first)
{
    return draft_rows(d, F, V, K, M, eps, hidden, NULL, 1, final_gamma, row_index, gamma, w_gate, w_up, w_down,
                      w_lm, conf, lse, token, margin, logits_out, hidden_out, conf_first, NULL, NULL);
}

/* Max-accept cap (Sec. 4.4): m = min(max(floor(0.7 n), 5), L). */
int mrp_oracle_cap(int n_masked, int L)
{
    int m = (int)floor(0.7 * (double)n_masked + 1e-9);
    if (m < 5) m = 5;
    if (m > L) m = L;
    return m;
}

/* Among candidate rows cand[0..n) pick the one with the largest confidence,
 * ties to the lower block position.  Returns its index into cand, or -1. */
static int best_candidate(const int *cand, int n, const uint8_t *taken, const float *c,
                          const int32_t *pos)
{
    int best = -1;
    for (int i = 0; i < n; ++i) {
        if (taken[i]) continue;
        if (best < 0) { best = i; continue; }
        const float ci = c[cand[i]], cb = c[cand[best]];
        if (ci > cb || (ci == cb && pos[cand[i]] < pos[cand[best]])) best = i;
    }
    return best;
}

/*
 * Reveal selection, remasking (Algorithms 2-4; Sec. 4.1 "Denoising Mode"; Sec. 4.4).
 *   conf  [(K+1), M] float32, token [(K+1), M] int32  -- per-step statistics of the masked rows
 *   row_index [M] or NULL: dense position b*L+i of each masked row (NULL = 0..M-1)
 *   mode 0 = STATIC: for k = 0..K take the r (k=0: r_reveal, k>=1: r_draft) most confident
 *            still-masked positions of each block under step k's logits; k=0 picks are
 *            reveals, k>=1 picks are drafts (listed in draft order).
 *   mode 1 = DYNAMIC + REMASK: R = {masked i : conf[0,i] >= tau}; if empty and
 *            ensure_progress, R = {most confident}; if use_cap and |R| > m keep the m most
 *            confident; remask i in R whose updated confidence c'(i) < tau, where
 *            c'(i) = min_{k=1..K} conf[k,i] (remask_policy 0) or conf[K,i] (policy 1);
 *            policy 2 follows the committed token instead of the top one: c'(i) =
 *            min_{k=1..K} conf_first[k,i], the probability the updated logits give the token
 *            revealed at step 0; policy 3 revokes i when the argmax moved away from that token
 *            at any step, token[k,i] != token[0,i] for some k in 1..K;
 *            if everything was revoked and ensure_progress, the most confident of R stays.
 *   conf_first [(K+1), M] float32: read by policy 2 only (NULL otherwise).
 * Outputs (all written for every dense position / block):
 *   reveal_mask, remask_mask [B*L] int8; out_token [B*L] int32 (-1 = nothing committed
 *   or drafted); step_of [B*L] int8 (-1 = untouched); draft_pos, draft_tok [B, Kd] int32
 *   (-1 pad) with Kd = K*r_draft; draft_len [B].
 * All confidence comparisons are float32 comparisons.
 */
int mrp_oracle_select(const float *conf, const int32_t *token, const int32_t *row_index,
                      int M, int K, int B, int L, int mode, float tau, int r_reveal,
                      int r_draft, int use_cap, int remask_policy, int ensure_progress,
                      int8_t *reveal_mask, int8_t *remask_mask, int32_t *out_token,
                      int8_t *step_of, int32_t *draft_pos, int32_t *draft_tok,
                      int32_t *draft_len, const float *conf_first)
{
    if (M < 0 || K < 0 || B <= 0 || L <= 0) return -1;
    if (mode == 1 && remask_policy == 2 && !conf_first) return -1;
    const int Kd = K * (r_draft > 0 ? r_draft : 0);
    for (int i = 0; i < B * L; ++i) {
        reveal_mask[i] = 0; remask_mask[i] = 0; out_token[i] = -1; step_of[i] = -1;
    }
    for (int i = 0; i < B * Kd; ++i) { draft_pos[i] = -1; draft_tok[i] = -1; }
    for (int b = 0; b < B; ++b) draft_len[b] = 0;

    int *cand = (int *)malloc(sizeof(int) * (size_t)(M > 0 ? M : 1));
    int32_t *pos = (int32_t *)malloc(sizeof(int32_t) * (size_t)(M > 0 ? M : 1));
    uint8_t *taken = (uint8_t *)malloc((size_t)(M > 0 ? M : 1));
    uint8_t *inR = (uint8_t *)malloc((size_t)(M > 0 ? M : 1));
    if (!cand || !pos || !taken || !inR) { free(cand); free(pos); free(taken); free(inR); return -1; }
    for (int m = 0; m < M; ++m) {
        const int idx = row_index ? row_index[m] : m;
        if (idx < 0 || idx >= B * L) { free(cand); free(pos); free(taken); free(inR); return -1; }
        pos[m] = idx % L;
    }

    for (int b = 0; b < B; ++b) {
        /* masked rows of this block */
        int n = 0;
        for (int m = 0; m < M; ++m) {
            const int idx = row_index ? row_index[m] : m;
            if (idx / L == b) cand[n++] = m;
        }
        if (n == 0) continue;
        memset(taken, 0, (size_t)n);

        if (mode == 0) {
            for (int k = 0; k <= K; ++k) {
                const int r = (k == 0) ? r_reveal : r_draft;
                const float *ck = conf + (size_t)k * M;
                for (int t = 0; t < r; ++t) {
                    const int bi = best_candidate(cand, n, taken, ck, pos);
                    if (bi < 0) break;
                    taken[bi] = 1;
                    const int m = cand[bi];
                    const int dense = b * L + pos[m];
                    out_token[dense] = token[(size_t)k * M + m];
                    step_of[dense] = (int8_t)k;
                    if (k == 0) {
                        reveal_mask[dense] = 1;
                    } else {
                        const int q = draft_len[b]++;
                        draft_pos[b * Kd + q] = pos[m];
                        draft_tok[b * Kd + q] = token[(size_t)k * M + m];
                    }
                }
            }
        } else {
            int nR = 0;
            for (int i = 0; i < n; ++i) { inR[i] = (conf[cand[i]] >= tau); nR += inR[i]; }
            if (nR == 0 && ensure_progress) {
                const int bi = best_candidate(cand, n, taken, conf, pos);
                inR[bi] = 1; nR = 1;
            }
            if (use_cap) {
                const int cap = mrp_oracle_cap(n, L);
                if (nR > cap) {
                    /* keep the cap most confident members of R */
                    for (int i = 0; i < n; ++i) taken[i] = !inR[i];
                    memset(inR, 0, (size_t)n);
                    for (int t = 0; t < cap; ++t) {
                        const int bi = best_candidate(cand, n, taken, conf, pos);
                        taken[bi] = 1; inR[bi] = 1;
                    }
                    nR = cap;
                    memset(taken, 0, (size_t)n);
                }
            }
            int kept = 0;
            for (int i = 0; i < n; ++i) {
                if (!inR[i]) continue;
                const int m = cand[i];
                const int dense = b * L + pos[m];
                reveal_mask[dense] = 1;
                int revoke;
                if (remask_policy == 3) {
                    revoke = 0;
                    for (int k = 1; k <= K; ++k)
                        if (token[(size_t)k * M + m] != token[m]) revoke = 1;
                } else {
                    const float *cu = (remask_policy == 2) ? conf_first : conf;
                    float c2;
                    if (K == 0) {
                        c2 = cu[m];
                    } else if (remask_policy == 1) {
                        c2 = cu[(size_t)K * M + m];
                    } else {
                        c2 = cu[(size_t)1 * M + m];
                        for (int k = 2; k <= K; ++k)
                            if (cu[(size_t)k * M + m] < c2) c2 = cu[(size_t)k * M + m];
                    }
                    revoke = (c2 < tau);
                }
                if (revoke) remask_mask[dense] = 1; else ++kept;
            }
            if (kept == 0 && nR > 0 && ensure_progress) {
                for (int i = 0; i < n; ++i) taken[i] = !inR[i];
                const int bi = best_candidate(cand, n, taken, conf, pos);
                remask_mask[b * L + pos[cand[bi]]] = 0;
            }
            for (int i = 0; i < n; ++i) {
                if (!inR[i]) continue;
                const int m = cand[i];
                const int dense = b * L + pos[m];
                if (!remask_mask[dense]) { out_token[dense] = token[m]; step_of[dense] = 0; }
            }
        }
    }
    free(cand); free(pos); free(taken); free(inR);
    return 0;
}

/*
 * Draft verification (Algorithm 3, rejection step: a drafted position is rejected where the
 * backbone's argmax differs from the draft; Figure 1(d): candidate k embeds the first k draft
 * tokens, hence prefix acceptance).
 *   draft_tok, verify_tok [B, Kd]; draft_len [B] (entries j >= draft_len[b] are ignored)
 *   positionwise = 0: accept_len = number of leading matches, accept_mask cleared after
 *                     the first mismatch (those drafts are remasked);
 *   positionwise = 1: accept_mask = per-slot match, accept_len = their count.
 */
int mrp_oracle_verify(const int32_t *draft_tok, const int32_t *verify_tok,
                      const int32_t *draft_len, int B, int Kd, int positionwise,
                      int32_t *accept_len, int8_t *accept_mask)
{
    if (B < 0 || Kd < 0) return -1;
    for (int b = 0; b < B; ++b) {
        int n = draft_len[b];
        if (n > Kd) n = Kd;
        if (n < 0) n = 0;
        int acc = 0, alive = 1;
        for (int j = 0; j < Kd; ++j) {
            int ok = (j < n) && (draft_tok[b * Kd + j] == verify_tok[b * Kd + j]);
            if (!positionwise) { if (!ok) alive = 0; ok = ok && alive; }
            accept_mask[b * Kd + j] = (int8_t)ok;
            acc += ok;
        }
        accept_len[b] = acc;
    }
    return 0;
}

/* ------------------------------------------------------------------------------------------------
 * The token-conditioned MRP module (Sec. 3.2; Fig. 1(a,c); Algorithm 2, "Delta, delta <- g(x_t, h)").
 *
 * One application of g to the L positions of each of B active blocks.  Sec. 3.2 fixes the parts --
 * the backbone's hidden states and the token embeddings of the (partly revealed) sequence, fused by a
 * learned projection; a small number D of transformer layers; the backbone's LM head on the result --
 * and leaves their details open.  The reading taken here (listed with the other readings in the
 * design notes):
 *     e_i = E[x_i]  (E the frozen embedding table; the [MASK] embedding where x_i = -1)
 *     z_i = W_p [h_i ; e_i]                                    (W_p [d, 2d], no bias)
 *     D times:  n = RMSNorm(z; g_attn);  q, k, v = W_q n, W_k n, W_v n;
 *               o_i = sum_j softmax_j(q_i . k_j / sqrt(d_head)) v_j   per attention head, j over the
 *                     positions of the same block (bidirectional, block-local, no positional term);
 *               z += W_o o;   n' = RMSNorm(z; g_mlp);   z += W_down( silu(W_gate n') * (W_up n') )
 *     Delta_i = z_i   (hidden residual),   delta_i = W_lm Delta_i   (logit residual)
 * Outputs: delta_h [B*L, d] double for every position; delta_l [M, V] double for the masked rows
 * listed in row_index (may be NULL with M = 0).  tokens [B*L] int32, -1 = masked.
 * Layer weights: arrays of D pointers each.  Returns 0, or -1 on bad arguments.
 *
 * The clean prefix (Fig. 1(c): the new block is decoded given the committed clean prefix, under the
 * same attention pattern as in training, where a block attends to itself and to the clean blocks in
 * front of it).  Reading: what a block sees of its prefix are the keys and values the module's own
 * layers produced for the prefix positions when those were committed; they are inputs here,
 * prefix_k / prefix_v = D pointers to [B, prefix_cap, d] arrays of which sequence b uses the first
 * prefix_len[b] rows (NULL = no prefix), and position i of block b attends to those rows and to the L
 * positions of its block in one softmax.  k_out / v_out (optional, D pointers to [B*L, d] doubles)
 * receive the keys and values of the block's own positions per layer: what a caller appends to the
 * prefix once the block is committed.
 */
int mrp_oracle_module_prefix(int d, int F, int V, int D, int n_attn_heads, int B, int L, int mask_token, double eps,
                             const float *hidden, const int32_t *tokens, const float *emb, const float *w_proj,
                             const float *const *g_attn, const float *const *w_q, const float *const *w_k,
                             const float *const *w_v, const float *const *w_o, const float *const *g_mlp,
                             const float *const *w_gate, const float *const *w_up, const float *const *w_down,
                             const float *w_lm, const int32_t *row_index, int M, double *delta_h, double *delta_l,
                             const float *const *prefix_k, const float *const *prefix_v, const int32_t *prefix_len,
                             int prefix_cap, double *const *k_out, double *const *v_out)
{
    if (d <= 0 || F <= 0 || V <= 0 || D < 0 || n_attn_heads <= 0 || d % n_attn_heads || B <= 0 || L <= 0) return -1;
    if (prefix_k && (!prefix_v || !prefix_len || prefix_cap < 0)) return -1;
    if (prefix_k)
        for (int b = 0; b < B; ++b)
            if (prefix_len[b] < 0 || prefix_len[b] > prefix_cap) return -1;
    const int dh = d / n_attn_heads;
    const size_t n = (size_t)B * L;
    const int max_keys = L + (prefix_k ? prefix_cap : 0);
    double *z = (double *)malloc(sizeof(double) * n * d), *nn = (double *)malloc(sizeof(double) * n * d);
    double *q = (double *)malloc(sizeof(double) * n * d), *k = (double *)malloc(sizeof(double) * n * d);
    double *v = (double *)malloc(sizeof(double) * n * d), *o = (double *)malloc(sizeof(double) * n * d);
    double *a = (double *)malloc(sizeof(double) * (size_t)F), *p = (double *)malloc(sizeof(double) * (size_t)max_keys);
    if (!z || !nn || !q || !k || !v || !o || !a || !p) { free(z); free(nn); free(q); free(k); free(v); free(o); free(a); free(p); return -1; }

    /* fusion of hidden state and token embedding */
    for (size_t i = 0; i < n; ++i) {
        const int tok = tokens[i] >= 0 ? tokens[i] : mask_token;
        const float *hi = hidden + i * (size_t)d, *ei = emb + (size_t)tok * d;
        for (int j = 0; j < d; ++j) {
            const float *wr = w_proj + (size_t)j * 2 * d;
            double s = 0.0;
            for (int c = 0; c < d; ++c) s += (double)wr[c] * (double)hi[c];
            for (int c = 0; c < d; ++c) s += (double)wr[d + c] * (double)ei[c];
            z[i * d + j] = s;
        }
    }
    for (int layer = 0; layer < D; ++layer) {
        /* attention sub-layer */
        for (size_t i = 0; i < n; ++i) {
            double ss = 0.0;
            for (int j = 0; j < d; ++j) ss += z[i * d + j] * z[i * d + j];
            const double rstd = 1.0 / sqrt(ss / (double)d + eps);
            for (int j = 0; j < d; ++j) nn[i * d + j] = z[i * d + j] * rstd * (double)g_attn[layer][j];
        }
        for (size_t i = 0; i < n; ++i)
            for (int j = 0; j < d; ++j) {
                double sq = 0.0, sk = 0.0, sv = 0.0;
                for (int c = 0; c < d; ++c) {
                    const double x = nn[i * d + c];
                    sq += (double)w_q[layer][(size_t)j * d + c] * x;
                    sk += (double)w_k[layer][(size_t)j * d + c] * x;
                    sv += (double)w_v[layer][(size_t)j * d + c] * x;
                }
                q[i * d + j] = sq; k[i * d + j] = sk; v[i * d + j] = sv;
            }
        if (k_out) memcpy(k_out[layer], k, sizeof(double) * n * d);
        if (v_out) memcpy(v_out[layer], v, sizeof(double) * n * d);
        for (int b = 0; b < B; ++b) {
            /* the keys of a position: the P_b rows of its sequence's clean prefix (Fig. 1(c)), then its block */
            const int P = prefix_k ? prefix_len[b] : 0;
            const float *pk = prefix_k ? prefix_k[layer] + (size_t)b * prefix_cap * d : NULL;
            const float *pv = prefix_k ? prefix_v[layer] + (size_t)b * prefix_cap * d : NULL;
            for (int hd = 0; hd < n_attn_heads; ++hd)
                for (int i = 0; i < L; ++i) {
                    const size_t ri = ((size_t)b * L + i) * d + (size_t)hd * dh;
                    double mx = -INFINITY;
                    for (int j = 0; j < P + L; ++j) {
                        double s = 0.0;
                        if (j < P) {
                            const float *kr = pk + (size_t)j * d + (size_t)hd * dh;
                            for (int c = 0; c < dh; ++c) s += q[ri + c] * (double)kr[c];
                        } else {
                            const size_t rj = ((size_t)b * L + (j - P)) * d + (size_t)hd * dh;
                            for (int c = 0; c < dh; ++c) s += q[ri + c] * k[rj + c];
                        }
                        p[j] = s / sqrt((double)dh);
                        if (p[j] > mx) mx = p[j];
                    }
                    double sum = 0.0;
                    for (int j = 0; j < P + L; ++j) { p[j] = exp(p[j] - mx); sum += p[j]; }
                    for (int c = 0; c < dh; ++c) {
                        double s = 0.0;
                        for (int j = 0; j < P; ++j) s += p[j] * (double)pv[(size_t)j * d + (size_t)hd * dh + c];
                        for (int j = 0; j < L; ++j) s += p[P + j] * v[((size_t)b * L + j) * d + (size_t)hd * dh + c];
                        o[ri + c] = s / sum;
                    }
                }
        }
        for (size_t i = 0; i < n; ++i)
            for (int j = 0; j < d; ++j) {
                double s = 0.0;
                for (int c = 0; c < d; ++c) s += (double)w_o[layer][(size_t)j * d + c] * o[i * d + c];
                nn[i * d + j] = s;                 /* held apart until every output of the row is done */
            }
        for (size_t i = 0; i < n * d; ++i) z[i] += nn[i];
        /* SwiGLU sub-layer */
        for (size_t i = 0; i < n; ++i) {
            double ss = 0.0;
            for (int j = 0; j < d; ++j) ss += z[i * d + j] * z[i * d + j];
            const double rstd = 1.0 / sqrt(ss / (double)d + eps);
            for (int j = 0; j < d; ++j) nn[i * d + j] = z[i * d + j] * rstd * (double)g_mlp[layer][j];
            for (int f = 0; f < F; ++f) {
                double g = 0.0, u = 0.0;
                for (int c = 0; c < d; ++c) {
                    g += (double)w_gate[layer][(size_t)f * d + c] * nn[i * d + c];
                    u += (double)w_up[layer][(size_t)f * d + c] * nn[i * d + c];
                }
                a[f] = g / (1.0 + exp(-g)) * u;
            }
            for (int j = 0; j < d; ++j) {
                double s = 0.0;
                for (int f = 0; f < F; ++f) s += (double)w_down[layer][(size_t)j * F + f] * a[f];
                q[i * d + j] = s;
            }
        }
        for (size_t i = 0; i < n * d; ++i) z[i] += q[i];
    }
    for (size_t i = 0; i < n * d; ++i) delta_h[i] = z[i];
    /* logit residual of the masked rows through the shared LM head */
    for (int m = 0; m < M; ++m) {
        const size_t row = row_index ? (size_t)row_index[m] : (size_t)m;
        if (row >= n) { free(z); free(nn); free(q); free(k); free(v); free(o); free(a); free(p); return -1; }
#pragma omp parallel for schedule(static)
        for (int t = 0; t < V; ++t) {
            double s = 0.0;
            for (int c = 0; c < d; ++c) s += (double)w_lm[(size_t)t * d + c] * z[row * d + c];
            delta_l[(size_t)m * V + t] = s;
        }
    }
    free(z); free(nn); free(q); free(k); free(v); free(o); free(a); free(p);
    return 0;
}

/* The module without a clean prefix: attention over the positions of the block alone. */
int mrp_oracle_module(int d, int F, int V, int D, int n_attn_heads, int B, int L, int mask_token, double eps,
                      const float *hidden, const int32_t *tokens, const float *emb, const float *w_proj,
                      const float *const *g_attn, const float *const *w_q, const float *const *w_k,
                      const float *const *w_v, const float *const *w_o, const float *const *g_mlp,
                      const float *const *w_gate, const float *const *w_up, const float *const *w_down,
                      const float *w_lm, const int32_t *row_index, int M, double *delta_h, double *delta_l)
{
    return mrp_oracle_module_prefix(d, F, V, D, n_attn_heads, B, L, mask_token, eps, hidden, tokens, emb, w_proj, g_attn, w_q,
                                    w_k, w_v, w_o, g_mlp, w_gate, w_up, w_down, w_lm, row_index, M, delta_h, delta_l, NULL, NULL,
                                    NULL, 0, NULL, NULL);
}
