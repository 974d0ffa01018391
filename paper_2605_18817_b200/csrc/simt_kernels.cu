// CUDA-core kernel family of the MRP drafting pass.
//
// This family computes everything in fp32 on the CUDA cores from fp32 or bf16 weights.  It is
// the production path of fp32 contexts (the tiny configuration), the path of bf16 shapes the
// tensor-core kernels do not cover, and an on-device cross-check of the tcgen05 family.
// Steps (Algorithm 2, inner loop): gather masked rows -> per head: RMSNorm, gate/up + SwiGLU,
// down projection and h <- h + Delta -> LM head on h_k - h_0 added to l_0 with per-slice
// softmax statistics -> combine over slices.
#include <float.h>
#include <limits.h>
#include <string.h>

#include <type_traits>

#include "mrp_internal.cuh"

namespace mrp {

__device__ __forceinline__ float ld_f(const float *p, size_t i) { return p[i]; }
__device__ __forceinline__ float ld_f(const __nv_bfloat16 *p, size_t i) { return __bfloat162float(p[i]); }

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

constexpr int kRC = 4;     // activation rows a warp handles per pass over a weight row

// Lane-partial dot products of one weight row with up to kRC activation rows (x: fp32 [rows, n_in]); the
// caller adds the lanes.  bf16 weight rows whose length is a multiple of 256 are read 16 bytes per lane.
template <typename T>
__device__ __forceinline__ void row_dots(const T *__restrict__ wr, const float *__restrict__ x, int rows, int n_in, int lane,
                                         float *s)
{
#pragma unroll
    for (int r = 0; r < kRC; ++r) s[r] = 0.f;
    if (std::is_same<T, __nv_bfloat16>::value && (n_in & 255) == 0) {
#pragma unroll 4
        for (int c = lane * 8; c < n_in; c += 256) {
            const uint4 q = __ldg(reinterpret_cast<const uint4 *>(reinterpret_cast<const __nv_bfloat16 *>(wr) + c));
            const float wv[8] = {__uint_as_float(q.x << 16), __uint_as_float(q.x & 0xFFFF0000u),
                                 __uint_as_float(q.y << 16), __uint_as_float(q.y & 0xFFFF0000u),
                                 __uint_as_float(q.z << 16), __uint_as_float(q.z & 0xFFFF0000u),
                                 __uint_as_float(q.w << 16), __uint_as_float(q.w & 0xFFFF0000u)};
#pragma unroll
            for (int r = 0; r < kRC; ++r) {
                if (r < rows) {
                    const float4 a = *reinterpret_cast<const float4 *>(x + (size_t)r * n_in + c);
                    const float4 b = *reinterpret_cast<const float4 *>(x + (size_t)r * n_in + c + 4);
                    float t = s[r];
                    t = fmaf(wv[0], a.x, t); t = fmaf(wv[1], a.y, t); t = fmaf(wv[2], a.z, t); t = fmaf(wv[3], a.w, t);
                    t = fmaf(wv[4], b.x, t); t = fmaf(wv[5], b.y, t); t = fmaf(wv[6], b.z, t); t = fmaf(wv[7], b.w, t);
                    s[r] = t;
                }
            }
        }
    } else {
        for (int c = lane; c < n_in; c += 32) {
            const float a = ld_f(wr, c);
#pragma unroll
            for (int r = 0; r < kRC; ++r)
                if (r < rows) s[r] = fmaf(a, x[(size_t)r * n_in + c], s[r]);
        }
    }
}

// ---- a0: gather masked rows into the fp32 residual stream --------------------------------
template <typename T>
__global__ void prep_kernel(const T *__restrict__ hidden, const int32_t *__restrict__ row_index,
                            int d, float *__restrict__ h0f, float *__restrict__ hcur, float *__restrict__ xt0,
                            const T *__restrict__ final_gamma, float eps, int n_rows_in,
                            int32_t *__restrict__ status, int32_t *__restrict__ user_status)
{
    pdl_trigger();
    pdl_wait();
    __shared__ float red[32];
    const int m = blockIdx.x;
    const int idx = row_index ? row_index[m] : m;
    // an index outside the caller's array is never used as an address: the row reads as zeros
    const bool bad = row_index && !row_ok(idx, n_rows_in);
    if (bad && threadIdx.x == 0) {
        atomicOr(status, MRP_DEV_BAD_INDEX);
        if (user_status) atomicOr(user_status, MRP_DEV_BAD_INDEX);
    }
    const size_t row = bad ? 0 : (size_t)idx;
    float ss = 0.f;
    for (int j = threadIdx.x; j < d; j += blockDim.x) {
        const float v = bad ? 0.f : ld_f(hidden, row * d + j);
        if (!xt0) h0f[(size_t)m * d + j] = v;
        hcur[(size_t)m * d + j] = v;
        ss = fmaf(v, v, ss);
    }
    if (!xt0) return;
    // No base logits: the LM-head operand of step 0 is n_0 = h_0, or RMSNorm(h_0) * final_gamma,
    // and h0f holds h_0 - n_0, so that the down projections emit n_0 + (h_k - h_0).
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float t = 0.f;
    for (int i = 0; i < (int)(blockDim.x >> 5); ++i) t += red[i];
    const float rstd0 = final_gamma ? rsqrtf(t / (float)d + eps) : 1.f;
    for (int j = threadIdx.x; j < d; j += blockDim.x) {
        const float v = bad ? 0.f : ld_f(hidden, row * d + j);
        const float n0 = final_gamma ? v * rstd0 * ld_f(final_gamma, j) : v;
        h0f[(size_t)m * d + j] = v - n0;
        xt0[(size_t)m * d + j] = n0;
    }
}

cudaError_t launch_prep(Ctx *c, const void *hidden, const int32_t *row_index, int M, cudaStream_t st, float *xt0,
                        int32_t *user_status)
{
    if (M == 0) return cudaSuccess;
    float *h0f = (float *)(c->ws + c->lay.h0f), *hcur = (float *)(c->ws + c->lay.hcur);
    int32_t *status = (int32_t *)(c->ws + c->lay.status);
    const bool pdl = !(c->cfg.flags & MRP_FLAG_NO_PDL);
    cudaError_t e;
    if (c->cfg.dtype == MRP_F32)
        e = launch_k(prep_kernel<float>, dim3(M), dim3(256), 0, st, pdl, (const float *)hidden, row_index, c->cfg.d, h0f, hcur,
                     xt0, (const float *)c->final_gamma, c->cfg.rms_eps, c->input_rows, status, user_status);
    else
        e = launch_k(prep_kernel<__nv_bfloat16>, dim3(M), dim3(256), 0, st, pdl, (const __nv_bfloat16 *)hidden, row_index,
                     c->cfg.d, h0f, hcur, xt0, (const __nv_bfloat16 *)c->final_gamma, c->cfg.rms_eps, c->input_rows,
                     status, user_status);
    c->launches++;
    return e;
}

// ---- a1: RMSNorm of the residual stream --------------------------------------------------
template <typename T>
__global__ void rmsnorm_kernel(const float *__restrict__ hcur, const T *__restrict__ gamma, int d,
                               float eps, float *__restrict__ xg)
{
    pdl_trigger();
    pdl_wait();
    __shared__ float red[32];
    const int m = blockIdx.x;
    const float *h = hcur + (size_t)m * d;
    float ss = 0.f;
    for (int j = threadIdx.x; j < d; j += blockDim.x) ss += h[j] * h[j];
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    if (threadIdx.x < 32) {
        float v = (threadIdx.x < (blockDim.x >> 5)) ? red[threadIdx.x] : 0.f;
        v = warp_sum(v);
        if (threadIdx.x == 0) red[0] = v;
    }
    __syncthreads();
    const float rstd = rsqrtf(red[0] / (float)d + eps);
    for (int j = threadIdx.x; j < d; j += blockDim.x)
        xg[(size_t)m * d + j] = h[j] * rstd * ld_f(gamma, j);
}

// ---- a1: gate/up projections + SwiGLU; one warp per inner feature, kRC rows at a time -------

template <typename T>
__global__ void gateup_kernel(const T *__restrict__ w_gate, const T *__restrict__ w_up,
                              const float *__restrict__ xg, int M, int d, int F,
                              float *__restrict__ act)
{
    pdl_trigger();
    pdl_wait();
    const int f = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (f >= F) return;
    const T *wg = w_gate + (size_t)f * d, *wu = w_up + (size_t)f * d;
    for (int m0 = 0; m0 < M; m0 += kRC) {
        float g[kRC], u[kRC];
        row_dots<T>(wg, xg + (size_t)m0 * d, M - m0, d, lane, g);
        row_dots<T>(wu, xg + (size_t)m0 * d, M - m0, d, lane, u);
#pragma unroll
        for (int r = 0; r < kRC; ++r) {
            const float gs = warp_sum(g[r]), us = warp_sum(u[r]);
            if (lane == 0 && m0 + r < M)
                act[(size_t)(m0 + r) * F + f] = gs / (1.f + expf(-gs)) * us;
        }
    }
}

// ---- a1: down projection, h <- h + Delta, LM-head operand h_k - h_0 ------------------------
template <typename T>
__global__ void down_kernel(const T *__restrict__ w_down, const float *__restrict__ act, int M,
                            int d, int F, float *__restrict__ hcur, const float *__restrict__ h0f,
                            float *__restrict__ xt_k, float *__restrict__ hidden_out)
{
    pdl_trigger();
    pdl_wait();
    const int j = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (j >= d) return;
    const T *wd = w_down + (size_t)j * F;
    for (int m0 = 0; m0 < M; m0 += kRC) {
        float s[kRC];
        row_dots<T>(wd, act + (size_t)m0 * F, M - m0, F, lane, s);
#pragma unroll
        for (int r = 0; r < kRC; ++r) {
            const float v = warp_sum(s[r]);
            if (lane == 0 && m0 + r < M) {
                const size_t o = (size_t)(m0 + r) * d + j;
                const float hn = hcur[o] + v;
                hcur[o] = hn;
                xt_k[o] = hn - h0f[o];
                if (hidden_out) hidden_out[o] = hn;
            }
        }
    }
}

// ---- a2 + a3: LM head on the residual, added to l_0, per-slice softmax statistics ---------
// A block owns vocabulary slices of SLICE (128, or 32 for small vocabularies) entries (grid-stride over slices).  For each
// chunk of kLR row-steps rs = k*M + m, the 8 warps compute delta for 16 entries each, the
// tile l = l_0 + delta goes to shared memory, and warp w reduces row-step w of the chunk.
constexpr int kLR = 8;

template <typename T, int SLICE>
__global__ void __launch_bounds__(256)
lm_simt_kernel(const T *__restrict__ w_lm, const float *__restrict__ xt, const float *__restrict__ xt0,
               const float *__restrict__ logits0, const int32_t *__restrict__ row_index, int M,
               int K, int d, int V, int n_slices, Partial *__restrict__ partials,
               float *__restrict__ logits_out, int n_rows_in, const float *__restrict__ teacher,
               KlPartial *__restrict__ kl_partials, int l0_bf16)
{
    pdl_trigger();
    pdl_wait();
    __shared__ float tile[kLR][SLICE];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_rs = (K + 1) * M;
    bool first = true;
    for (int slice = blockIdx.x; slice < n_slices; slice += gridDim.x, first = false) {
        const int v0 = slice * SLICE;
        for (int rs0 = 0; rs0 < n_rs; rs0 += kLR) {
            // delta for entries v0 + warp*16 .. +16, row-steps rs0 .. rs0+kLR
            for (int e = 0; e < SLICE / 8; ++e) {
                const int vl = warp * (SLICE / 8) + e;
                const int v = v0 + vl;
                float acc[kLR];
#pragma unroll
                for (int r = 0; r < kLR; ++r) acc[r] = 0.f;
                if (v < V) {
                    const T *wr = w_lm + (size_t)v * d;
                    for (int j = lane; j < d; j += 32) {
                        const float a = ld_f(wr, j);
#pragma unroll
                        for (int r = 0; r < kLR; ++r) {
                            const int rs = rs0 + r;
                            if (rs < n_rs && rs >= M)   // step 0 has no residual ...
                                acc[r] = fmaf(a, xt[(size_t)(rs - M) * d + j], acc[r]);
                            else if (rs < M && xt0)     // ... unless its logits are computed here
                                acc[r] = fmaf(a, xt0[(size_t)rs * d + j], acc[r]);
                        }
                    }
                }
#pragma unroll
                for (int r = 0; r < kLR; ++r) {
                    const float s = warp_sum(acc[r]);
                    const int rs = rs0 + r;
                    if (lane == 0) {
                        float l = -INFINITY;
                        if (v < V && rs < n_rs) {
                            const int m = rs % M;
                            const int idx = row_index ? row_index[m] : m;
                            const bool have = logits0 && (!row_index || row_ok(idx, n_rows_in));
                            l = (have ? ld_l0(logits0, l0_bf16, (size_t)idx * (size_t)V + v) : 0.f) + s;
                        }
                        tile[r][vl] = l;
                    }
                }
            }
            __syncthreads();
            const int rs = rs0 + warp;
            if (rs < n_rs) {
                float mx = -INFINITY, sec = -INFINITY;
                int idx = INT_MAX;
                float vals[SLICE / 32];
#pragma unroll
                for (int i = 0; i < SLICE / 32; ++i) {
                    const int vl = lane + 32 * i;
                    const float l = tile[warp][vl];
                    vals[i] = l;
                    if (l > mx) { sec = mx; mx = l; idx = v0 + vl; }
                    else if (l > sec) sec = l;
                }
                if (mx == -INFINITY) idx = INT_MAX;
                // warp merge of (mx, idx, second)
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    const float omx = __shfl_xor_sync(0xffffffffu, mx, o);
                    const int oidx = __shfl_xor_sync(0xffffffffu, idx, o);
                    const float osec = __shfl_xor_sync(0xffffffffu, sec, o);
                    const bool ow = (omx > mx) || (omx == mx && oidx < idx);
                    const float lo = ow ? mx : omx;
                    float ns = lo > sec ? lo : sec;
                    ns = osec > ns ? osec : ns;
                    sec = ns;
                    if (ow) { mx = omx; idx = oidx; }
                }
                float sum = 0.f;
#pragma unroll
                for (int i = 0; i < SLICE / 32; ++i)
                    sum += (vals[i] == -INFINITY) ? 0.f : expf(vals[i] - mx);
                sum = warp_sum(sum);
                if (logits_out && rs >= M) {
#pragma unroll
                    for (int i = 0; i < SLICE / 32; ++i) {
                        const int v = v0 + lane + 32 * i;
                        if (v < V) logits_out[(size_t)(rs - M) * V + v] = vals[i];
                    }
                }
                if (lane == 0) {
                    Partial p;
                    p.mx = mx; p.sum = sum; p.idx = idx; p.second = sec;
                    Partial *dst = partials + (size_t)blockIdx.x * n_rs + rs;
                    if (!first) p = merge_partial(*dst, p);
                    *dst = p;
                }
                if (teacher && rs >= M) {
                    // the slice's share of the KL objective against the teacher logits of this row-step
                    const float *tr = teacher + (size_t)(rs - M) * V;
                    float tv[SLICE / 32], tmx = -INFINITY;
#pragma unroll
                    for (int i = 0; i < SLICE / 32; ++i) {
                        const int v = v0 + lane + 32 * i;
                        tv[i] = v < V ? tr[v] : -INFINITY;
                        tmx = fmaxf(tmx, tv[i]);
                    }
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) tmx = fmaxf(tmx, __shfl_xor_sync(0xffffffffu, tmx, o));
                    float ts = 0.f, tc = 0.f;
#pragma unroll
                    for (int i = 0; i < SLICE / 32; ++i) {
                        if (tv[i] != -INFINITY) {
                            const float e = expf(tv[i] - tmx);
                            ts += e;
                            tc = fmaf(e, tv[i] - vals[i], tc);
                        }
                    }
                    ts = warp_sum(ts);
                    tc = warp_sum(tc);
                    if (lane == 0) {
                        KlPartial q;
                        q.mx = tmx; q.sum = ts; q.cross = tc; q.pad = 0.f;
                        KlPartial *dst = kl_partials + (size_t)blockIdx.x * (size_t)(K * M) + (rs - M);
                        if (!first) q = merge_kl(*dst, q);
                        *dst = q;
                    }
                }
            }
            __syncthreads();
        }
    }
}

// ---- a4: combine per-slice partials -------------------------------------------------------
__global__ void combine_kernel(const Partial *__restrict__ partials, int n_slices, int n_rs,
                               float *__restrict__ conf, float *__restrict__ lse,
                               int32_t *__restrict__ token, float *__restrict__ margin,
                               int32_t *__restrict__ status, int32_t *__restrict__ user_status,
                               const TopFix fix, const KlPartial *__restrict__ kl_partials, int M,
                               float *__restrict__ kl_out)
{
    pdl_trigger();
    pdl_wait();
    const int rs = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (rs >= n_rs) return;
    Partial p;
    p.mx = -INFINITY; p.sum = 0.f; p.idx = INT_MAX; p.second = -INFINITY;
#pragma unroll 8
    for (int s = lane; s < n_slices; s += 32) p = merge_partial(p, partials[(size_t)s * n_rs + rs]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        Partial q;
        q.mx = __shfl_xor_sync(0xffffffffu, p.mx, o);
        q.sum = __shfl_xor_sync(0xffffffffu, p.sum, o);
        q.idx = __shfl_xor_sync(0xffffffffu, p.idx, o);
        q.second = __shfl_xor_sync(0xffffffffu, p.second, o);
        // fixed operand order (lower lane first) keeps the result identical on both sides
        p = (lane & o) ? merge_partial(q, p) : merge_partial(p, q);
    }
    float top = p.mx;      // the top logit as the sum of exponentials saw it
    const bool has_operand = fix.xt && (rs >= fix.M || !fix.logits0);   // step 0 of mrp_draft has none
    float ssq = 0.f;       // sum of squares of the row-step's LM-head operand (hi part)
    if (fix.w && has_operand) {
        // exact top logit: l_0[row, tok] + W[tok] . (hi + lo), fp32, fixed summation order
        // (no l_0 term, and step 0 included, when the base logits are computed in the pass)
        const int tok = __shfl_sync(0xffffffffu, p.idx, 0);
        const int m = rs % fix.M;
        const int idx = fix.row_index ? fix.row_index[m] : m;
        const bool have = fix.logits0 && (!fix.row_index || row_ok(idx, fix.n_rows_in));
        const __nv_bfloat16 *wr = fix.w + (size_t)tok * fix.d;
        const __nv_bfloat16 *xh = fix.xt + (size_t)rs * fix.d, *xl = xh + (size_t)fix.n_rs * fix.d;
        float dot = 0.f;
#pragma unroll 8
        for (int j = lane * 2; j < fix.d; j += 64) {
            const float2 w2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(wr + j));
            const float2 h2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(xh + j));
            const float2 l2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(xl + j));
            dot = fmaf(w2.x, h2.x + l2.x, dot);
            dot = fmaf(w2.y, h2.y + l2.y, dot);
            ssq = fmaf(h2.x, h2.x, fmaf(h2.y, h2.y, ssq));
        }
        dot = warp_sum(dot);
        top = (have ? ld_l0(fix.logits0, fix.l0_bf16, (size_t)idx * (size_t)fix.V + tok) : 0.f) + dot;
    } else if (fix.range_limit > 0.f && has_operand) {
        // only the size of the operand row is needed: 16-byte loads of its hi part (d % 64 == 0)
        const uint4 *xh = reinterpret_cast<const uint4 *>(fix.xt + (size_t)rs * fix.d);
#pragma unroll 4
        for (int j = lane; j < fix.d / 8; j += 32) {
            const uint4 q = xh[j];
            const uint32_t w4[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 h2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&w4[i]));
                ssq = fmaf(h2.x, h2.x, fmaf(h2.y, h2.y, ssq));
            }
        }
    }
    if (fix.range_limit > 0.f && has_operand) {
        // accuracy range of the tensor-core path: d * rms(operand row) = sqrt(d * sum of squares)
        ssq = warp_sum(ssq);
        if (lane == 0 && sqrtf(ssq * (float)fix.d) > fix.range_limit) {
            atomicOr(status, MRP_DEV_RANGE);
            if (user_status) atomicOr(user_status, MRP_DEV_RANGE);
        }
    }
    KlPartial kq;
    kq.mx = -INFINITY; kq.sum = 0.f; kq.cross = 0.f; kq.pad = 0.f;
    if (kl_out && rs >= M) {
        // KL objective of the row-step: merge the slices' partial sums in the same fixed order
        const size_t n_kl = (size_t)(n_rs - M);
#pragma unroll 4
        for (int s = lane; s < n_slices; s += 32) kq = merge_kl(kq, kl_partials[(size_t)s * n_kl + (rs - M)]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            KlPartial q;
            q.mx = __shfl_xor_sync(0xffffffffu, kq.mx, o);
            q.sum = __shfl_xor_sync(0xffffffffu, kq.sum, o);
            q.cross = __shfl_xor_sync(0xffffffffu, kq.cross, o);
            q.pad = 0.f;
            kq = (lane & o) ? merge_kl(q, kq) : merge_kl(kq, q);
        }
    }
    if (lane == 0) {
        // the term of the top token entered the sum as exp(0) = 1: swap in its exact value
        const float sum = (top == p.mx) ? p.sum : (p.sum - 1.f) + expf(top - p.mx);
        const float l = p.mx + logf(sum);
        if (kl_out && rs >= M) kl_out[rs - M] = kq.cross / kq.sum - (kq.mx + logf(kq.sum)) + l;
        conf[rs] = (top == p.mx) ? 1.f / sum : expf(top - l);
        lse[rs] = l;
        token[rs] = p.idx;
        if (margin) margin[rs] = top - p.second;
        if (!isfinite(l)) {
            atomicOr(status, MRP_DEV_NONFINITE);
            if (user_status) atomicOr(user_status, MRP_DEV_NONFINITE);
        }
    }
}

cudaError_t launch_combine(Ctx *c, const Partial *partials, int n_slices, int n_rowsteps,
                           const mrp_draft_out &out, int32_t *status, cudaStream_t st, const TopFix *fix, int M)
{
    if (n_rowsteps == 0) return cudaSuccess;
    const int warps = 4;
    TopFix f;
    memset(&f, 0, sizeof(f));
    if (fix) f = *fix;
    c->launches++;
    return launch_k(combine_kernel, dim3((n_rowsteps + warps - 1) / warps), dim3(warps * 32), 0, st,
                    !(c->cfg.flags & MRP_FLAG_NO_PDL), partials, n_slices, n_rowsteps, out.conf, out.lse,
                    out.token, out.margin, status, out.status, f,
                    (const KlPartial *)(c->teacher ? c->ws + c->lay.kl_partials : nullptr), M,
                    c->teacher ? c->kl_out : (float *)nullptr);
}

// ---- conf_first: probability of the step-0 argmax token under every step's logits ----------
__global__ void first_token_prob_kernel(const FirstTok f, const int32_t *__restrict__ token,
                                        const float *__restrict__ lse, const float *__restrict__ conf,
                                        float *__restrict__ conf_first)
{
    pdl_trigger();
    pdl_wait();
    const int rs = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (rs >= (f.K + 1) * f.M) return;
    const int k = rs / f.M, m = rs - k * f.M;
    if (k == 0) {                     // the step-0 token is the top token of step 0
        if (lane == 0) conf_first[rs] = conf[rs];
        return;
    }
    const int tok = token[m];
    float dot = 0.f;
    if (f.x_bf16 && f.w8_scale) {
        // 8-bit LM head: the row of the dequantised matrix, scale[tok] * e4m3 code
        const __nv_bfloat16 *xh = (const __nv_bfloat16 *)f.x + (size_t)rs * f.d;
        const __nv_bfloat16 *xl = xh + (size_t)f.lo_rows * f.d;
        const uint8_t *wr = (const uint8_t *)f.w + (size_t)tok * f.d;
        for (int j = lane; j < f.d; j += 32) {
            const uint32_t b = wr[j];
            const int e = (b >> 3) & 15, mm = b & 7;
            float wv = e ? __uint_as_float(((uint32_t)(e + 120) << 23) | ((uint32_t)mm << 20)) : (float)mm * 0.001953125f;
            wv = (b & 0x80u) ? -wv : wv;
            dot = fmaf(wv, __bfloat162float(xh[j]) + __bfloat162float(xl[j]), dot);
        }
        dot *= f.w8_scale[tok];
    } else if (f.x_bf16) {
        const __nv_bfloat16 *xh = (const __nv_bfloat16 *)f.x + (size_t)rs * f.d;
        const __nv_bfloat16 *xl = xh + (size_t)f.lo_rows * f.d;
        const __nv_bfloat16 *wr = (const __nv_bfloat16 *)f.w + (size_t)tok * f.d;
        for (int j = lane; j < f.d; j += 32)
            dot = fmaf(__bfloat162float(wr[j]), __bfloat162float(xh[j]) + __bfloat162float(xl[j]), dot);
    } else {
        // the row of step k holds h_k - h_0, or n_0 + h_k - h_0 when the base logits are computed in the pass
        const float *xr = (const float *)f.x + (size_t)(k - 1) * f.M * f.d + (size_t)m * f.d;
        for (int j = lane; j < f.d; j += 32) {
            const float wv = f.w_bf16 ? __bfloat162float(((const __nv_bfloat16 *)f.w)[(size_t)tok * f.d + j])
                                      : ((const float *)f.w)[(size_t)tok * f.d + j];
            dot = fmaf(wv, xr[j], dot);
        }
    }
    dot = warp_sum(dot);
    if (lane == 0) {
        const int idx = f.row_index ? f.row_index[m] : m;
        const bool have = f.logits0 && (!f.row_index || row_ok(idx, f.n_rows_in));
        const float l = (have ? ld_l0(f.logits0, f.l0_bf16, (size_t)idx * (size_t)f.V + tok) : 0.f) + dot;
        conf_first[rs] = fminf(expf(l - lse[rs]), conf[rs]);     // never above the top probability
    }
}

cudaError_t launch_first_token_prob(Ctx *c, const FirstTok &f, const mrp_draft_out &out, cudaStream_t st)
{
    if (!out.conf_first) return cudaSuccess;
    const int n = (f.K + 1) * f.M, warps = 4;
    c->launches++;
    return launch_k(first_token_prob_kernel, dim3((n + warps - 1) / warps), dim3(warps * 32), 0, st,
                    !(c->cfg.flags & MRP_FLAG_NO_PDL), f, (const int32_t *)out.token, (const float *)out.lse,
                    (const float *)out.conf, out.conf_first);
}

template <typename T>
static cudaError_t simt_lm_tail_t(Ctx *c, const float *logits0, const int32_t *row_index, int M, int K,
                                  const mrp_draft_out &out, cudaStream_t st)
{
    const int d = c->cfg.d, V = c->cfg.vocab;
    float *xt = (float *)(c->ws + c->lay.xt);
    Partial *partials = (Partial *)(c->ws + c->lay.partials);
    KlPartial *kl_partials = (KlPartial *)(c->ws + c->lay.kl_partials);
    int32_t *status = (int32_t *)(c->ws + c->lay.status);
    const bool pdl = !(c->cfg.flags & MRP_FLAG_NO_PDL);
    float *xt0 = c->from_hidden ? xt + (size_t)K * M * d : nullptr;
    cudaError_t e;
    prof_mark(c, 1, st);
    e = note_err(c, wait_logits0(c, st), "wait for the base logits");
    if (e != cudaSuccess) return e;
    // small vocabularies: narrower slices so that every SM gets a block
    const bool narrow = (V + kSimtSliceV - 1) / kSimtSliceV < 2 * c->sm_count;
    const int slice_v = narrow ? 32 : kSimtSliceV;
    const int n_slices = (V + slice_v - 1) / slice_v;
    const int grid = n_slices < kSimtMaxBlocks ? n_slices : kSimtMaxBlocks;
    if (narrow)
        e = launch_k(lm_simt_kernel<T, 32>, dim3(grid), dim3(256), 0, st, pdl, (const T *)c->w_lm, (const float *)xt,
                     (const float *)xt0, logits0, row_index, M, K, d, V, n_slices, partials, out.logits_out,
                     c->input_rows, c->teacher, kl_partials, c->l0_bf16 ? 1 : 0);
    else
        e = launch_k(lm_simt_kernel<T, kSimtSliceV>, dim3(grid), dim3(256), 0, st, pdl, (const T *)c->w_lm,
                     (const float *)xt, (const float *)xt0, logits0, row_index, M, K, d, V, n_slices, partials,
                     out.logits_out, c->input_rows, c->teacher, kl_partials, c->l0_bf16 ? 1 : 0);
    c->launches++;
    if (e != cudaSuccess) return e;
    prof_mark(c, 2, st);
    e = launch_combine(c, partials, grid, (K + 1) * M, out, status, st, nullptr, M);
    prof_mark(c, 3, st);
    if (e != cudaSuccess) return e;
    FirstTok ft;
    memset(&ft, 0, sizeof(ft));
    ft.w = c->w_lm; ft.w_bf16 = c->cfg.dtype == MRP_BF16; ft.logits0 = logits0; ft.row_index = row_index;
    ft.l0_bf16 = c->l0_bf16 ? 1 : 0;
    ft.n_rows_in = c->input_rows; ft.x = xt; ft.x_bf16 = 0; ft.M = M; ft.K = K; ft.d = d; ft.V = V;
    return launch_first_token_prob(c, ft, out, st);
}

cudaError_t simt_lm_tail(Ctx *c, const float *logits0, const int32_t *row_index, int M, int K,
                         const mrp_draft_out &out, cudaStream_t st)
{
    if (c->cfg.dtype == MRP_F32) return simt_lm_tail_t<float>(c, logits0, row_index, M, K, out, st);
    return simt_lm_tail_t<__nv_bfloat16>(c, logits0, row_index, M, K, out, st);
}

template <typename T>
static cudaError_t simt_draft_t(Ctx *c, const void *hidden, const float *logits0,
                                const int32_t *row_index, int M, int K, const mrp_draft_out &out,
                                cudaStream_t st)
{
    const int d = c->cfg.d, F = c->cfg.d_ff, V = c->cfg.vocab;
    float *h0f = (float *)(c->ws + c->lay.h0f), *hcur = (float *)(c->ws + c->lay.hcur);
    float *xg = (float *)(c->ws + c->lay.xg), *act = (float *)(c->ws + c->lay.act);
    float *xt = (float *)(c->ws + c->lay.xt);
    Partial *partials = (Partial *)(c->ws + c->lay.partials);
    KlPartial *kl_partials = (KlPartial *)(c->ws + c->lay.kl_partials);
    int32_t *status = (int32_t *)(c->ws + c->lay.status);
    const bool pdl = !(c->cfg.flags & MRP_FLAG_NO_PDL);
    prof_mark(c, 0, st);
    // without base logits the operand rows of step 0 (n_0) follow those of steps 1..K
    float *xt0 = c->from_hidden ? xt + (size_t)K * M * d : nullptr;
    cudaError_t e = launch_prep(c, hidden, row_index, M, st, xt0, out.status);
    if (e != cudaSuccess) return e;
    if (K == 0 && out.hidden_out)
        cudaMemcpyAsync(out.hidden_out, hcur, sizeof(float) * (size_t)M * d, cudaMemcpyDeviceToDevice, st);
    for (int k = 1; k <= K; ++k) {
        const mrp_head_weights &hw = c->heads[k - 1];
        e = launch_k(rmsnorm_kernel<T>, dim3(M), dim3(256), 0, st, pdl, (const float *)hcur, (const T *)hw.rms_gamma, d,
                     c->cfg.rms_eps, xg);
        if (e == cudaSuccess)
            e = launch_k(gateup_kernel<T>, dim3((F + 7) / 8), dim3(256), 0, st, pdl, (const T *)hw.w_gate,
                         (const T *)hw.w_up, (const float *)xg, M, d, F, act);
        if (e == cudaSuccess)
            e = launch_k(down_kernel<T>, dim3((d + 7) / 8), dim3(256), 0, st, pdl, (const T *)hw.w_down,
                         (const float *)act, M, d, F, hcur, (const float *)h0f, xt + (size_t)(k - 1) * M * d,
                         (k == K) ? out.hidden_out : (float *)nullptr);
        if (e != cudaSuccess) return e;
        c->launches += 3;
    }
    return simt_lm_tail(c, logits0, row_index, M, K, out, st);
}

cudaError_t simt_draft(Ctx *c, const void *hidden, const float *logits0, const int32_t *row_index,
                       int M, int K, const mrp_draft_out &out, cudaStream_t st)
{
    if (M == 0) return cudaSuccess;
    if (c->cfg.dtype == MRP_F32)
        return simt_draft_t<float>(c, hidden, logits0, row_index, M, K, out, st);
    return simt_draft_t<__nv_bfloat16>(c, hidden, logits0, row_index, M, K, out, st);
}

// ---------------------------------------------------------------------------------------
// The token-conditioned MRP module (Sec. 3.2; Algorithm 2, "Delta, delta <- g(x_t, h)") on CUDA cores.
// fp32 activations, weights in the context's dtype.  One step = embedding fusion, D transformer layers
// with block-local attention, h <- h + Delta, the LM-head operand h - h_0 of the masked rows, and then the
// context's own LM-head kernels.
// ---------------------------------------------------------------------------------------
// [h_i ; emb[x_i]] per dense position; a token outside the table reads as masked and raises the bit.
template <typename T>
__global__ void mod_concat_kernel(const float *h_state, const T *__restrict__ hidden0, int first_step,
                                  const int32_t *__restrict__ tokens, const T *__restrict__ emb, int mask_token,
                                  int emb_rows, int d, float *h_out /* = h_state */, float *__restrict__ cat,
                                  int32_t *__restrict__ status, int32_t *__restrict__ user_status)
{
    pdl_trigger();
    pdl_wait();
    const int i = blockIdx.x;
    int tok = tokens[i];
    if (tok >= emb_rows || tok < -1) {
        if (threadIdx.x == 0) {
            atomicOr(status, MRP_DEV_BAD_INDEX);
            if (user_status) atomicOr(user_status, MRP_DEV_BAD_INDEX);
        }
        tok = -1;
    }
    if (tok < 0) tok = mask_token;
    for (int j = threadIdx.x; j < d; j += blockDim.x) {
        const float h = first_step ? ld_f(hidden0, (size_t)i * d + j) : h_state[(size_t)i * d + j];
        if (first_step) h_out[(size_t)i * d + j] = h;
        cat[(size_t)i * 2 * d + j] = h;
        cat[(size_t)i * 2 * d + d + j] = ld_f(emb, (size_t)tok * d + j);
    }
}

// y[r, j] (+)= sum_c W[j, c] x[r, c]: one warp per output feature, kRC rows at a time; bf16 weights
// with n_in a multiple of 256 are read 16 bytes per lane.
template <typename T>
__global__ void linear_kernel(const T *__restrict__ w, const float *__restrict__ x, int rows, int n_in, int n_out,
                              float *__restrict__ y, int accumulate)
{
    pdl_trigger();
    pdl_wait();
    const int j = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (j >= n_out) return;
    const T *wr = w + (size_t)j * n_in;
    for (int r0 = 0; r0 < rows; r0 += kRC) {
        float s[kRC];
        row_dots<T>(wr, x + (size_t)r0 * n_in, rows - r0, n_in, lane, s);
#pragma unroll
        for (int r = 0; r < kRC; ++r) {
            const float v = warp_sum(s[r]);
            if (lane == 0 && r0 + r < rows) {
                const size_t o = (size_t)(r0 + r) * n_out + j;
                y[o] = accumulate ? y[o] + v : v;
            }
        }
    }
}

// Block-local bidirectional attention: CTA = (block b, attention head); a warp per query position, lanes
// over the key positions for the scores and over the head's features for the output.
__global__ void mod_attention_kernel(const float *__restrict__ q, const float *__restrict__ k,
                                     const float *__restrict__ v, int L, int d, int dh, float *__restrict__ o)
{
    pdl_trigger();
    pdl_wait();
    extern __shared__ float prob[];                  // [warps][L]
    const int b = blockIdx.x, hd = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = blockDim.x >> 5;
    float *p = prob + (size_t)warp * L;
    const float scale = rsqrtf((float)dh);
    for (int i = warp; i < L; i += n_warps) {
        const float *qi = q + ((size_t)b * L + i) * d + (size_t)hd * dh;
        float mx = -INFINITY;
        for (int j = lane; j < L; j += 32) {
            const float *kj = k + ((size_t)b * L + j) * d + (size_t)hd * dh;
            float sdot = 0.f;
            for (int c = 0; c < dh; ++c) sdot = fmaf(qi[c], kj[c], sdot);
            sdot *= scale;
            p[j] = sdot;
            mx = fmaxf(mx, sdot);
        }
#pragma unroll
        for (int w = 16; w > 0; w >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, w));
        float sum = 0.f;
        for (int j = lane; j < L; j += 32) {
            const float e = expf(p[j] - mx);
            p[j] = e;
            sum += e;
        }
        sum = warp_sum(sum);
        __syncwarp();
        for (int c = lane; c < dh; c += 32) {
            float acc = 0.f;
            for (int j = 0; j < L; ++j) acc = fmaf(p[j], v[((size_t)b * L + j) * d + (size_t)hd * dh + c], acc);
            o[((size_t)b * L + i) * d + (size_t)hd * dh + c] = acc / sum;
        }
        __syncwarp();
    }
}

// h <- h + Delta for every dense position.
__global__ void mod_add_kernel(float *__restrict__ h_state, const float *__restrict__ z, size_t n)
{
    pdl_trigger();
    pdl_wait();
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
        h_state[i] += z[i];
}

// LM-head operand of the masked rows: h - h_0, as the context's kernel family wants it (fp32 rows for the
// CUDA-core family; bf16 hi + lo rows of step 1 behind zero rows of step 0, plus the fp16 copy when the
// row-major fp16 LM head runs, for the tensor-core family).
template <typename T>
__global__ void mod_operand_kernel(const float *__restrict__ h_state, const T *__restrict__ hidden0,
                                   const int32_t *__restrict__ row_index, int n_rows_in, int M, int d,
                                   float *__restrict__ xt_f32, __nv_bfloat16 *__restrict__ xt_bf16, int lo_rows,
                                   __half *__restrict__ xt16, float *__restrict__ hidden_out,
                                   int32_t *__restrict__ status, int32_t *__restrict__ user_status)
{
    pdl_trigger();
    pdl_wait();
    const int m = blockIdx.x;
    const int idx = row_index ? row_index[m] : m;
    const bool bad = !row_ok(idx, n_rows_in);
    if (bad && threadIdx.x == 0) {
        atomicOr(status, MRP_DEV_BAD_INDEX);
        if (user_status) atomicOr(user_status, MRP_DEV_BAD_INDEX);
    }
    for (int j = threadIdx.x; j < d; j += blockDim.x) {
        const float h = bad ? 0.f : h_state[(size_t)idx * d + j];
        const float r = bad ? 0.f : h - ld_f(hidden0, (size_t)idx * d + j);
        if (hidden_out) hidden_out[(size_t)m * d + j] = h;
        if (xt_f32) xt_f32[(size_t)m * d + j] = r;
        if (xt_bf16) {
            const __nv_bfloat16 hi = __float2bfloat16_rn(r);
            xt_bf16[(size_t)m * d + j] = __float2bfloat16(0.f);                          // step 0 has no residual
            xt_bf16[((size_t)lo_rows + m) * d + j] = __float2bfloat16(0.f);
            xt_bf16[((size_t)M + m) * d + j] = hi;
            xt_bf16[((size_t)lo_rows + M + m) * d + j] = __float2bfloat16_rn(r - __bfloat162float(hi));
            if (xt16) xt16[(size_t)m * d + j] = __float2half_rn(r);
        }
    }
}

size_t module_workspace_bytes(const mrp_config &cfg, int n_layers)
{
    (void)n_layers;
    const size_t n = (size_t)cfg.max_seqs * cfg.block_len, d = (size_t)cfg.d, F = (size_t)cfg.d_ff;
    return align_up(n * 2 * d * 4, 256) + 6 * align_up(n * d * 4, 256) + align_up(n * F * 4, 256);
}

template <typename T>
static cudaError_t module_step_t(Ctx *c, const int32_t *tokens, const void *hidden0, float *h_state, const float *logits0,
                                 const int32_t *row_index, int M, int B, int L, bool first_step, const mrp_draft_out &out,
                                 cudaStream_t st)
{
    const mrp_module_weights &w = c->module;
    const int d = c->cfg.d, F = c->cfg.d_ff, n = B * L, dh = d / w.n_attn_heads;
    const size_t cap = (size_t)c->cfg.max_seqs * c->cfg.block_len;
    char *ws = c->module_ws;
    auto take = [&](size_t bytes) { char *p0 = ws; ws += align_up(bytes, 256); return (float *)p0; };
    float *cat = take(cap * 2 * d * 4), *z = take(cap * d * 4), *nn = take(cap * d * 4), *q = take(cap * d * 4);
    float *k = take(cap * d * 4), *v = take(cap * d * 4), *o = take(cap * d * 4), *act = take(cap * F * 4);
    int32_t *status = (int32_t *)(c->ws + c->lay.status);
    const bool pdl = !(c->cfg.flags & MRP_FLAG_NO_PDL);
    auto lin = [&](const void *wm, const float *x, int n_in, int n_out, float *y, int acc) {
        c->launches++;
        return launch_k(linear_kernel<T>, dim3((n_out + 7) / 8), dim3(256), 0, st, pdl, (const T *)wm, x, n, n_in, n_out, y, acc);
    };
    prof_mark(c, 0, st);
    cudaError_t e = launch_k(mod_concat_kernel<T>, dim3(n), dim3(256), 0, st, pdl, (const float *)h_state, (const T *)hidden0,
                             first_step ? 1 : 0, tokens, (const T *)w.emb, w.mask_token, w.emb_rows, d, h_state, cat, status,
                             out.status);
    c->launches++;
    if (e == cudaSuccess) e = lin(w.w_proj, cat, 2 * d, d, z, 0);
    for (int l = 0; l < w.n_layers && e == cudaSuccess; ++l) {
        const mrp_module_layer &y = w.layers[l];
        e = launch_k(rmsnorm_kernel<T>, dim3(n), dim3(256), 0, st, pdl, (const float *)z, (const T *)y.g_attn, d, c->cfg.rms_eps, nn);
        c->launches++;
        if (e == cudaSuccess) e = lin(y.w_q, nn, d, d, q, 0);
        if (e == cudaSuccess) e = lin(y.w_k, nn, d, d, k, 0);
        if (e == cudaSuccess) e = lin(y.w_v, nn, d, d, v, 0);
        if (e == cudaSuccess) {
            e = launch_k(mod_attention_kernel, dim3(B, w.n_attn_heads), dim3(128), (size_t)4 * L * 4, st, pdl, (const float *)q,
                         (const float *)k, (const float *)v, L, d, dh, o);
            c->launches++;
        }
        if (e == cudaSuccess) e = lin(y.w_o, o, d, d, z, 1);
        if (e == cudaSuccess) {
            e = launch_k(rmsnorm_kernel<T>, dim3(n), dim3(256), 0, st, pdl, (const float *)z, (const T *)y.g_mlp, d, c->cfg.rms_eps, nn);
            c->launches++;
        }
        if (e == cudaSuccess) {
            e = launch_k(gateup_kernel<T>, dim3((F + 7) / 8), dim3(256), 0, st, pdl, (const T *)y.w_gate, (const T *)y.w_up,
                         (const float *)nn, n, d, F, act);
            c->launches++;
        }
        if (e == cudaSuccess) e = lin(y.w_down, act, F, d, z, 1);
    }
    if (e == cudaSuccess) {
        const size_t total = (size_t)n * d;
        e = launch_k(mod_add_kernel, dim3((unsigned)((total + 255) / 256 < 1184 ? (total + 255) / 256 : 1184)), dim3(256), 0, st, pdl,
                     h_state, (const float *)z, total);
        c->launches++;
    }
    if (e != cudaSuccess || M == 0) return e;
    // the LM-head operand of the masked rows, then the context's LM-head kernels (K = 1)
    if (c->use_tc) {
        const TcPlan pl = tc_plan(c, M, 1, out, st, false);
        __nv_bfloat16 *xt = (__nv_bfloat16 *)(c->ws + c->lay.xt);
        e = launch_k(mod_operand_kernel<T>, dim3(M), dim3(256), 0, st, pdl, (const float *)h_state, (const T *)hidden0, row_index,
                     n, M, d, (float *)nullptr, xt, c->lo_xt, pl.f16_lm ? (__half *)(c->ws + c->lay.xt16) : (__half *)nullptr,
                     out.hidden_out, status, out.status);
        c->launches++;
        if (e != cudaSuccess) return e;
        return tc_lm_tail(c, pl, logits0, row_index, M, 1, out, st);
    }
    e = launch_k(mod_operand_kernel<T>, dim3(M), dim3(256), 0, st, pdl, (const float *)h_state, (const T *)hidden0, row_index, n,
                 M, d, (float *)(c->ws + c->lay.xt), (__nv_bfloat16 *)nullptr, 0, (__half *)nullptr, out.hidden_out, status,
                 out.status);
    c->launches++;
    if (e != cudaSuccess) return e;
    return simt_lm_tail(c, logits0, row_index, M, 1, out, st);
}

cudaError_t module_step(Ctx *c, const int32_t *tokens, const void *hidden0, float *h_state, const float *logits0,
                        const int32_t *row_index, int M, int B, int L, bool first_step, const mrp_draft_out &out,
                        cudaStream_t st)
{
    if (c->cfg.dtype == MRP_F32)
        return module_step_t<float>(c, tokens, hidden0, h_state, logits0, row_index, M, B, L, first_step, out, st);
    return module_step_t<__nv_bfloat16>(c, tokens, hidden0, h_state, logits0, row_index, M, B, L, first_step, out, st);
}

}  // namespace mrp
