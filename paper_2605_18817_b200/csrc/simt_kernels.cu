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

#include <atomic>
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

// Loads of buffers that another CTA of the SAME kernel may have written in an earlier phase (the one-kernel
// pass below): CG = true reads through L2 (ld.global.cg), never from a line this SM cached before the write.
template <bool CG> __device__ __forceinline__ float ldx(const float *p) { return CG ? __ldcg(p) : *p; }
template <bool CG> __device__ __forceinline__ float4 ldx4(const float *p)
{
    return CG ? __ldcg(reinterpret_cast<const float4 *>(p)) : *reinterpret_cast<const float4 *>(p);
}
template <bool CG> __device__ __forceinline__ int ldxi(const int32_t *p) { return CG ? __ldcg(p) : *p; }
template <bool CG> __device__ __forceinline__ Partial ld_partial(const Partial *p)
{
    if (!CG) return *p;
    const float4 q = __ldcg(reinterpret_cast<const float4 *>(p));
    Partial r;
    r.mx = q.x; r.sum = q.y; r.idx = __float_as_int(q.z); r.second = q.w;
    return r;
}

// Lane-partial dot products of one weight row with up to kRC activation rows (x: fp32 [rows, n_in]); the
// caller adds the lanes.  bf16 weight rows whose length is a multiple of 256 are read 16 bytes per lane.
template <typename T, bool CG = false>
__device__ __forceinline__ void row_dots(const T *__restrict__ wr, const float *x, int rows, int n_in, int lane,
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
                    const float4 a = ldx4<CG>(x + (size_t)r * n_in + c);
                    const float4 b = ldx4<CG>(x + (size_t)r * n_in + c + 4);
                    float t = s[r];
                    t = fmaf(wv[0], a.x, t); t = fmaf(wv[1], a.y, t); t = fmaf(wv[2], a.z, t); t = fmaf(wv[3], a.w, t);
                    t = fmaf(wv[4], b.x, t); t = fmaf(wv[5], b.y, t); t = fmaf(wv[6], b.z, t); t = fmaf(wv[7], b.w, t);
                    s[r] = t;
                }
            }
        }
    } else {
#pragma unroll 8
        for (int c = lane; c < n_in; c += 32) {
            const float a = ld_f(wr, c);
#pragma unroll
            for (int r = 0; r < kRC; ++r)
                if (r < rows) s[r] = fmaf(a, ldx<CG>(x + (size_t)r * n_in + c), s[r]);
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

// The work of CTA `cta` of `n_cta` (256 threads); `tile` is kLR * SLICE floats of its shared memory.
template <typename T, int SLICE>
__device__ __forceinline__ void
lm_simt_body(float (*tile)[SLICE], int cta, int n_cta,
             const T *__restrict__ w_lm, const float *__restrict__ xt, const float *__restrict__ xt0,
             const float *__restrict__ logits0, const int32_t *__restrict__ row_index, int M,
             int K, int d, int V, int n_slices, Partial *__restrict__ partials,
             float *__restrict__ logits_out, int n_rows_in, const float *__restrict__ teacher,
             KlPartial *__restrict__ kl_partials, int l0_bf16)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_rs = (K + 1) * M;
    bool first = true;
    for (int slice = cta; slice < n_slices; slice += n_cta, first = false) {
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
                    Partial *dst = partials + (size_t)cta * n_rs + rs;
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
                        KlPartial *dst = kl_partials + (size_t)cta * (size_t)(K * M) + (rs - M);
                        if (!first) q = merge_kl(*dst, q);
                        *dst = q;
                    }
                }
            }
            __syncthreads();
        }
    }
}

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
    lm_simt_body<T, SLICE>(tile, blockIdx.x, gridDim.x, w_lm, xt, xt0, logits0, row_index, M, K, d, V, n_slices, partials,
                           logits_out, n_rows_in, teacher, kl_partials, l0_bf16);
}

// ---- a4: combine per-slice partials -------------------------------------------------------
// One warp merges the slices of row-step rs.
template <bool CG = false>
__device__ __forceinline__ void combine_body(int rs, int lane, const Partial *partials, int n_slices, int n_rs,
                                             float *__restrict__ conf, float *__restrict__ lse,
                                             int32_t *__restrict__ token, float *__restrict__ margin,
                                             int32_t *__restrict__ status, int32_t *__restrict__ user_status,
                                             const TopFix &fix, const KlPartial *__restrict__ kl_partials, int M,
                                             float *__restrict__ kl_out)
{
    Partial p;
    p.mx = -INFINITY; p.sum = 0.f; p.idx = INT_MAX; p.second = -INFINITY;
#pragma unroll 8
    for (int s = lane; s < n_slices; s += 32) p = merge_partial(p, ld_partial<CG>(partials + (size_t)s * n_rs + rs));
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
        // (the base logit of the top token is asked for before the dot product, not after it)
        const float l0_top = have ? ld_l0(fix.logits0, fix.l0_bf16, (size_t)idx * (size_t)fix.V + tok) : 0.f;
        float dot = 0.f;
        if ((fix.d & 255) == 0) {
            // 16 bytes per lane and load: the three rows of a step of 256 elements are in flight together
#pragma unroll 8
            for (int j = lane * 8; j < fix.d; j += 256) {
                const uint4 wq = __ldg(reinterpret_cast<const uint4 *>(wr + j));
                const uint4 hq = *reinterpret_cast<const uint4 *>(xh + j);
                const uint4 lq = *reinterpret_cast<const uint4 *>(xl + j);
                const uint32_t w4[4] = {wq.x, wq.y, wq.z, wq.w}, h4[4] = {hq.x, hq.y, hq.z, hq.w}, l4[4] = {lq.x, lq.y, lq.z, lq.w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float2 w2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&w4[i]));
                    const float2 h2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&h4[i]));
                    const float2 l2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&l4[i]));
                    dot = fmaf(w2.x, h2.x + l2.x, dot);
                    dot = fmaf(w2.y, h2.y + l2.y, dot);
                    ssq = fmaf(h2.x, h2.x, fmaf(h2.y, h2.y, ssq));
                }
            }
        } else {
#pragma unroll 8
            for (int j = lane * 2; j < fix.d; j += 64) {
                const float2 w2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(wr + j));
                const float2 h2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(xh + j));
                const float2 l2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(xl + j));
                dot = fmaf(w2.x, h2.x + l2.x, dot);
                dot = fmaf(w2.y, h2.y + l2.y, dot);
                ssq = fmaf(h2.x, h2.x, fmaf(h2.y, h2.y, ssq));
            }
        }
        dot = warp_sum(dot);
        top = l0_top + dot;
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
    if (rs >= n_rs) return;
    combine_body(rs, threadIdx.x & 31, partials, n_slices, n_rs, conf, lse, token, margin, status, user_status, fix,
                 kl_partials, M, kl_out);
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
template <bool CG = false>
__device__ __forceinline__ void first_token_prob_body(int rs, int lane, const FirstTok &f, const int32_t *token,
                                                      const float *lse, const float *conf, float *conf_first)
{
    const int k = rs / f.M, m = rs - k * f.M;
    if (k == 0) {                     // the step-0 token is the top token of step 0
        if (lane == 0) conf_first[rs] = ldx<CG>(conf + rs);
        return;
    }
    const int tok = ldxi<CG>(token + m);
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
            dot = fmaf(wv, ldx<CG>(xr + j), dot);
        }
    }
    dot = warp_sum(dot);
    if (lane == 0) {
        const int idx = f.row_index ? f.row_index[m] : m;
        const bool have = f.logits0 && (!f.row_index || row_ok(idx, f.n_rows_in));
        const float l = (have ? ld_l0(f.logits0, f.l0_bf16, (size_t)idx * (size_t)f.V + tok) : 0.f) + dot;
        conf_first[rs] = fminf(expf(l - ldx<CG>(lse + rs)), ldx<CG>(conf + rs));     // never above the top probability
    }
}

__global__ void first_token_prob_kernel(const FirstTok f, const int32_t *__restrict__ token,
                                        const float *__restrict__ lse, const float *__restrict__ conf,
                                        float *__restrict__ conf_first)
{
    pdl_trigger();
    pdl_wait();
    const int rs = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (rs >= (f.K + 1) * f.M) return;
    first_token_prob_body(rs, threadIdx.x & 31, f, token, lse, conf, conf_first);
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

// ---- the whole pass as ONE kernel, for a few short rows ---------------------------------------
// A small shape (the tiny configuration: 4 rows of 256) is a dozen launches of a few microseconds each when
// every step is a kernel of its own; here the same steps are phases of one cooperative kernel, separated by
// grid barriers: gather -> per head [RMSNorm + gate/up + SwiGLU | down projection + residual] -> LM head with
// per-CTA softmax partials -> combine -> (probability of the step-0 token).  The phases run the code of the
// separate kernels (row_dots, lm_simt_body, combine_body), reading what earlier phases wrote through L2.
// The barrier is a counter that only grows: a launch reads where the last one left it (bar[1]), barrier i
// is passed once the counter reaches base + (i + 1) * gridDim.x, and CTA 0 leaves base + n_barriers *
// gridDim.x behind for the next launch.  A wait that runs out (about half a second) raises MRP_DEV_TIMEOUT,
// and the CTA adds the arrivals it still owes before it returns, so that the counter ends where the next
// launch expects it whatever happened.
constexpr int kFusedMaxRows = 8;
constexpr int kFusedMaxD = 512;
constexpr int kFusedMaxHeads = 8;
constexpr int kFusedMaxRowSteps = 32;  // (K + 1) * M: a lane per row-step in the LM-head phase
constexpr int kFusedEntries = 4;       // vocabulary entries a warp works on at a time in the LM-head phase
constexpr size_t kFusedMaxSmem = 160 * 1024;
constexpr long long kFusedBarrierCycles = 1000000000LL;

template <typename T>
struct FusedParams {
    const T *hidden, *w_lm, *final_gamma;
    const T *gamma[kFusedMaxHeads], *w_gate[kFusedMaxHeads], *w_up[kFusedMaxHeads], *w_down[kFusedMaxHeads];
    const int32_t *row_index;
    const float *logits0;
    int M, K, d, F, V, n_rows_in, l0_bf16;
    float eps;
    float *h0f, *hcur, *act, *xt, *xt0;     // workspace (xt0: operand rows of step 0, or nullptr)
    Partial *partials;
    float *conf, *lse, *margin, *logits_out, *hidden_out, *conf_first;
    int32_t *token;
    int32_t *status, *user_status;
    unsigned int *bar;                      // [0] arrivals so far, [1] their number when this launch began
    FirstTok ft;
};

struct FusedSync {
    unsigned int base;
    int done, total;
};

// All threads of all CTAs.  False: the wait ran out (the caller returns; the owed arrivals are already paid).
template <typename P>
__device__ __forceinline__ bool fused_barrier(const P &p, FusedSync &sy)
{
    __syncthreads();
    int ok = 1;
    sy.done++;
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(p.bar, 1u);
        const unsigned int target = sy.base + (unsigned int)sy.done * gridDim.x;
        const long long t0 = clock64();
        while ((int)(*reinterpret_cast<volatile unsigned int *>(p.bar) - target) < 0) {
            if (clock64() - t0 > kFusedBarrierCycles) { ok = 0; break; }
        }
        __threadfence();
        if (!ok) {
            atomicOr(p.status, MRP_DEV_TIMEOUT);
            if (p.user_status) atomicOr(p.user_status, MRP_DEV_TIMEOUT);
            if (sy.total > sy.done) atomicAdd(p.bar, (unsigned int)(sy.total - sy.done));
        }
    }
    return __syncthreads_and(ok) != 0;
}

template <typename T>
__global__ void __launch_bounds__(256)
simt_fused_kernel(const FusedParams<T> p)
{
    // normalised rows [M, d] in the head phases; in the LM-head phase the operand rows [(K+1) M, d + 1],
    // one weight row per warp [8, d] and the warps' partials [8, 32]
    extern __shared__ __align__(16) float sh[];
    __shared__ float red[8];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = gridDim.x, cta = blockIdx.x;
    const int gw = cta * 8 + warp, n_gw = G * 8;
    const int M = p.M, K = p.K, d = p.d, F = p.F;
    FusedSync sy;
    sy.base = *reinterpret_cast<volatile unsigned int *>(p.bar + 1);
    sy.done = 0;
    sy.total = 2 * K + 3 + (p.conf_first ? 1 : 0);
    // what CTA 0 leaves for the next launch, on every way out
    auto leave = [&]() {
        if (cta == 0 && threadIdx.x == 0) {
            *reinterpret_cast<volatile unsigned int *>(p.bar + 1) = sy.base + (unsigned int)sy.total * G;
            __threadfence();
        }
    };

    // ---- gather the masked rows (CTA per row) ----
    for (int m = cta; m < M; m += G) {
        const int idx = p.row_index ? p.row_index[m] : m;
        const bool bad = p.row_index && !row_ok(idx, p.n_rows_in);
        if (bad && threadIdx.x == 0) {
            atomicOr(p.status, MRP_DEV_BAD_INDEX);
            if (p.user_status) atomicOr(p.user_status, MRP_DEV_BAD_INDEX);
        }
        const size_t row = bad ? 0 : (size_t)idx;
        float ss = 0.f;
        for (int j = threadIdx.x; j < d; j += blockDim.x) {
            const float v = bad ? 0.f : ld_f(p.hidden, row * d + j);
            if (!p.xt0) p.h0f[(size_t)m * d + j] = v;
            p.hcur[(size_t)m * d + j] = v;
            ss = fmaf(v, v, ss);
        }
        if (p.xt0) {
            // no base logits: step 0's operand is n_0 = h_0 or RMSNorm(h_0) * final_gamma, h0f = h_0 - n_0
            ss = warp_sum(ss);
            __syncthreads();
            if (lane == 0) red[warp] = ss;
            __syncthreads();
            float t = 0.f;
            for (int i = 0; i < 8; ++i) t += red[i];
            const float rstd0 = p.final_gamma ? rsqrtf(t / (float)d + p.eps) : 1.f;
            for (int j = threadIdx.x; j < d; j += blockDim.x) {
                const float v = bad ? 0.f : ld_f(p.hidden, row * d + j);
                const float n0 = p.final_gamma ? v * rstd0 * ld_f(p.final_gamma, j) : v;
                p.h0f[(size_t)m * d + j] = v - n0;
                p.xt0[(size_t)m * d + j] = n0;
            }
        }
    }
    if (!fused_barrier(p, sy)) { leave(); return; }

    for (int k = 1; k <= K; ++k) {
        // ---- RMSNorm of all rows into shared memory (every CTA its own copy), then gate/up + SwiGLU ----
        for (int m = warp; m < M; m += 8) {
            float ss = 0.f;
#pragma unroll 8
            for (int j = lane; j < d; j += 32) {
                const float v = __ldcg(p.hcur + (size_t)m * d + j);
                sh[m * d + j] = v;
                ss = fmaf(v, v, ss);
            }
            ss = warp_sum(ss);
            const float rstd = rsqrtf(ss / (float)d + p.eps);
            for (int j = lane; j < d; j += 32) sh[m * d + j] = sh[m * d + j] * rstd * ld_f(p.gamma[k - 1], j);
        }
        __syncthreads();
        for (int f = gw; f < F; f += n_gw) {
            const T *wg = p.w_gate[k - 1] + (size_t)f * d, *wu = p.w_up[k - 1] + (size_t)f * d;
            for (int m0 = 0; m0 < M; m0 += kRC) {
                float g[kRC], u[kRC];
                row_dots<T>(wg, sh + (size_t)m0 * d, M - m0, d, lane, g);
                row_dots<T>(wu, sh + (size_t)m0 * d, M - m0, d, lane, u);
#pragma unroll
                for (int r = 0; r < kRC; ++r) {
                    const float gs = warp_sum(g[r]), us = warp_sum(u[r]);
                    if (lane == 0 && m0 + r < M) p.act[(size_t)(m0 + r) * F + f] = gs / (1.f + expf(-gs)) * us;
                }
            }
        }
        if (!fused_barrier(p, sy)) { leave(); return; }
        // ---- down projection, h <- h + Delta, LM-head operand h_k - h_0 ----
        if (cta * 8 < d) {             // CTAs with an output feature: the activations [M, F] into shared memory, through L2
            for (int i = threadIdx.x * 4; i < M * F; i += blockDim.x * 4) {
                if (((M * F) & 3) == 0) *reinterpret_cast<float4 *>(sh + i) = __ldcg(reinterpret_cast<const float4 *>(p.act + i));
                else for (int e = i; e < i + 4 && e < M * F; ++e) sh[e] = __ldcg(p.act + e);
            }
        }
        __syncthreads();
        for (int j = gw; j < d; j += n_gw) {
            const T *wd = p.w_down[k - 1] + (size_t)j * F;
            for (int m0 = 0; m0 < M; m0 += kRC) {
                float s[kRC];
                row_dots<T>(wd, sh + (size_t)m0 * F, M - m0, F, lane, s);
#pragma unroll
                for (int r = 0; r < kRC; ++r) {
                    const float v = warp_sum(s[r]);
                    if (lane == 0 && m0 + r < M) {
                        const size_t o = (size_t)(m0 + r) * d + j;
                        const float hn = __ldcg(p.hcur + o) + v;
                        p.hcur[o] = hn;
                        p.xt[(size_t)(k - 1) * M * d + o] = hn - __ldcg(p.h0f + o);
                        if (k == K && p.hidden_out) p.hidden_out[o] = hn;
                    }
                }
            }
        }
        if (!fused_barrier(p, sy)) { leave(); return; }
    }

    // ---- LM head on the residuals, added to l_0 (Eq. 2), softmax statistics per CTA ----
    // Lane = row-step: a warp takes one vocabulary entry at a time, puts its weight row into shared memory,
    // and every lane forms the whole dot product of its own operand row with it; the lane then folds the logit
    // into the running statistics of its row-step, so nothing is exchanged between lanes until the end.
    const int n_rs = (K + 1) * M;
    {
        const int ldx_s = d + 1;                       // odd pitch: lanes read one column of 32 rows without conflicts
        const size_t xs_floats = ((size_t)n_rs * ldx_s + 3) & ~(size_t)3;
        const size_t w_floats = ((size_t)8 * kFusedEntries * d + 3) & ~(size_t)3;
        float *xs = sh, *wrow = sh + xs_floats + (size_t)warp * kFusedEntries * d;
        Partial *wp = reinterpret_cast<Partial *>(sh + xs_floats + w_floats);
        const bool vec = (d & 3) == 0;                 // 16-byte reads of the (broadcast) weight rows
        if (vec) {
#pragma unroll 4
            for (int i = threadIdx.x * 4; i < n_rs * d; i += blockDim.x * 4) {
                const int rs = i / d, j = i - rs * d;
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);              // step 0 has no residual ...
                if (rs >= M) v = __ldcg(reinterpret_cast<const float4 *>(p.xt + (size_t)(rs - M) * d + j));
                else if (p.xt0) v = __ldcg(reinterpret_cast<const float4 *>(p.xt0 + (size_t)rs * d + j));   // ... unless computed here
                float *dst = xs + rs * ldx_s + j;
                dst[0] = v.x; dst[1] = v.y; dst[2] = v.z; dst[3] = v.w;
            }
        } else {
#pragma unroll 4
            for (int i = threadIdx.x; i < n_rs * d; i += blockDim.x) {
                const int rs = i / d, j = i - rs * d;
                float v = 0.f;
                if (rs >= M) v = __ldcg(p.xt + (size_t)(rs - M) * d + j);
                else if (p.xt0) v = __ldcg(p.xt0 + (size_t)rs * d + j);
                xs[rs * ldx_s + j] = v;
            }
        }
        __syncthreads();
        Partial st;
        st.mx = -INFINITY; st.sum = 0.f; st.idx = INT_MAX; st.second = -INFINITY;
        const bool mine = lane < n_rs;
        const int m = mine ? lane % M : 0;
        const int idx = p.row_index ? p.row_index[m] : m;
        const bool have = mine && p.logits0 && (!p.row_index || row_ok(idx, p.n_rows_in));
        const float *xr = xs + (size_t)(mine ? lane : 0) * ldx_s;
        // kFusedEntries consecutive entries per warp and round: every operand element read from shared memory
        // feeds that many products
        for (int v0 = gw * kFusedEntries; v0 < p.V; v0 += n_gw * kFusedEntries) {
            const int n_e = min(kFusedEntries, p.V - v0);
            float l0[kFusedEntries];
#pragma unroll
            for (int e = 0; e < kFusedEntries; ++e)
                l0[e] = (have && e < n_e) ? ld_l0(p.logits0, p.l0_bf16, (size_t)idx * (size_t)p.V + v0 + e) : 0.f;
#pragma unroll 8
            for (int i = lane; i < n_e * d; i += 32) wrow[i] = ld_f(p.w_lm, (size_t)v0 * d + i);
            for (int i = n_e * d + lane; i < kFusedEntries * d; i += 32) wrow[i] = 0.f;
            __syncwarp();
            // two running sums per entry, each over every other group of four (short chains keep the fp32
            // rounding of a long dot product small)
            float a[kFusedEntries][2];
#pragma unroll
            for (int e = 0; e < kFusedEntries; ++e) a[e][0] = a[e][1] = 0.f;
            int j = 0;
            if (vec) {
                for (; j + 8 <= d; j += 8) {
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const float x0 = xr[j + 4 * h], x1 = xr[j + 4 * h + 1], x2 = xr[j + 4 * h + 2], x3 = xr[j + 4 * h + 3];
#pragma unroll
                        for (int e = 0; e < kFusedEntries; ++e) {
                            const float4 w4 = *reinterpret_cast<const float4 *>(wrow + e * d + j + 4 * h);
                            float t = a[e][h];
                            t = fmaf(w4.x, x0, t); t = fmaf(w4.y, x1, t); t = fmaf(w4.z, x2, t); t = fmaf(w4.w, x3, t);
                            a[e][h] = t;
                        }
                    }
                }
            }
            for (; j < d; ++j) {
                const float x0 = xr[j];
#pragma unroll
                for (int e = 0; e < kFusedEntries; ++e) a[e][0] = fmaf(wrow[e * d + j], x0, a[e][0]);
            }
            __syncwarp();
            if (mine) {
#pragma unroll
                for (int e = 0; e < kFusedEntries; ++e) {
                    if (e < n_e) {
                        const int v = v0 + e;
                        const float l = l0[e] + (a[e][0] + a[e][1]);
                        if (l > st.mx) {                 // entries come in ascending order: the lowest id keeps a tie
                            st.sum = st.sum * expf(st.mx - l) + 1.f;
                            st.second = st.mx; st.mx = l; st.idx = v;
                        } else {
                            st.sum += expf(l - st.mx);
                            if (l > st.second) st.second = l;
                        }
                        if (p.logits_out && lane >= M) p.logits_out[(size_t)(lane - M) * p.V + v] = l;
                    }
                }
            }
        }
        wp[warp * 32 + lane] = st;
        __syncthreads();
        if (warp == 0 && mine) {
            Partial t = wp[lane];
#pragma unroll
            for (int w8 = 1; w8 < 8; ++w8) t = merge_partial(t, wp[w8 * 32 + lane]);
            p.partials[(size_t)cta * n_rs + lane] = t;
        }
    }
    if (!fused_barrier(p, sy)) { leave(); return; }

    // ---- combine the CTAs' partials (warp per row-step) ----
    const int n_parts = G;
    TopFix nofix;
    memset(&nofix, 0, sizeof(nofix));
    for (int rs = gw; rs < n_rs; rs += n_gw)
        combine_body<true>(rs, lane, p.partials, n_parts, n_rs, p.conf, p.lse, p.token, p.margin, p.status, p.user_status,
                           nofix, nullptr, M, nullptr);
    if (p.conf_first) {
        if (!fused_barrier(p, sy)) { leave(); return; }
        for (int rs = gw; rs < n_rs; rs += n_gw)
            first_token_prob_body<true>(rs, lane, p.ft, p.token, p.lse, p.conf, p.conf_first);
    }
    // the last barrier: nobody leaves (and CTA 0 does not publish the next base) before all have arrived
    fused_barrier(p, sy);
    leave();
}

static size_t fused_smem(int M, int K, int d)
{
    const size_t lm = ((((size_t)(K + 1) * M * (d + 1) + 3) & ~(size_t)3) + (((size_t)8 * kFusedEntries * d + 3) & ~(size_t)3)) * 4 +
                      8 * 32 * sizeof(Partial);
    return lm;      // (the head phases' [M, d] and [M, F] arrays are checked against it in fused_ok)
}

// Whether a call runs as the one-kernel pass: a few short rows, at least one head, no KL objective; not under
// MRP_FLAG_NO_CHAIN (which asks for one kernel per step).
static bool fused_ok(const Ctx *c, int M, int K)
{
    return M >= 1 && M <= kFusedMaxRows && c->cfg.d <= kFusedMaxD && K >= 1 && K <= kFusedMaxHeads &&
           (K + 1) * M <= kFusedMaxRowSteps && !c->teacher && !(c->cfg.flags & MRP_FLAG_NO_CHAIN) &&
           fused_smem(M, K, c->cfg.d) <= kFusedMaxSmem && (size_t)M * c->cfg.d_ff * 4 <= fused_smem(M, K, c->cfg.d);
}

template <typename T>
static cudaError_t simt_fused_t(Ctx *c, const void *hidden, const float *logits0, const int32_t *row_index, int M, int K,
                                const mrp_draft_out &out, cudaStream_t st, bool *launched)
{
    *launched = false;
    auto kern = simt_fused_kernel<T>;
    // all CTAs wait for one another: they must be resident together (asked once per device)
    static std::atomic<unsigned long long> asked{0}, fits{0};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const unsigned long long bit = 1ull << (dev & 63);
    if (!(asked.load() & bit)) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kFusedMaxSmem);
        if (e != cudaSuccess) return e;
        int per_sm = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, 256, kFusedMaxSmem);
        if (e != cudaSuccess) return e;
        if (per_sm >= 1) fits.fetch_or(bit);
        asked.fetch_or(bit);
    }
    if (!(fits.load() & bit)) return cudaSuccess;
    const int d = c->cfg.d, V = c->cfg.vocab;
    FusedParams<T> p;
    memset(&p, 0, sizeof(p));
    p.hidden = (const T *)hidden; p.w_lm = (const T *)c->w_lm; p.final_gamma = (const T *)c->final_gamma;
    for (int k = 0; k < K; ++k) {
        p.gamma[k] = (const T *)c->heads[k].rms_gamma; p.w_gate[k] = (const T *)c->heads[k].w_gate;
        p.w_up[k] = (const T *)c->heads[k].w_up; p.w_down[k] = (const T *)c->heads[k].w_down;
    }
    p.row_index = row_index; p.logits0 = logits0;
    p.M = M; p.K = K; p.d = d; p.F = c->cfg.d_ff; p.V = V; p.n_rows_in = c->input_rows; p.l0_bf16 = c->l0_bf16 ? 1 : 0;
    p.eps = c->cfg.rms_eps;
    p.h0f = (float *)(c->ws + c->lay.h0f); p.hcur = (float *)(c->ws + c->lay.hcur);
    p.act = (float *)(c->ws + c->lay.act); p.xt = (float *)(c->ws + c->lay.xt);
    p.xt0 = c->from_hidden ? p.xt + (size_t)K * M * d : nullptr;
    p.partials = (Partial *)(c->ws + c->lay.partials);
    p.conf = out.conf; p.lse = out.lse; p.margin = out.margin; p.logits_out = out.logits_out; p.hidden_out = out.hidden_out;
    p.conf_first = out.conf_first; p.token = out.token;
    p.status = (int32_t *)(c->ws + c->lay.status); p.user_status = out.status;
    p.bar = (unsigned int *)(c->ws + c->lay.status) + 16;
    p.ft.w = c->w_lm; p.ft.w_bf16 = c->cfg.dtype == MRP_BF16; p.ft.logits0 = logits0; p.ft.row_index = row_index;
    p.ft.l0_bf16 = p.l0_bf16; p.ft.n_rows_in = c->input_rows; p.ft.x = p.xt; p.ft.x_bf16 = 0;
    p.ft.M = M; p.ft.K = K; p.ft.d = d; p.ft.V = V;
    int grid = c->sm_count;
    if (grid > c->lay.n_slices_max) grid = c->lay.n_slices_max;
    prof_mark(c, 0, st);
    e = note_err(c, wait_logits0(c, st), "wait for the base logits");
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(256);
    cfg.dynamicSmemBytes = fused_smem(M, K, d);
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeCooperative;
    at[0].val.cooperative = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, kern, p);
    if (e == cudaErrorCooperativeLaunchTooLarge) {
        // the context may use fewer SMs than the device has (MPS share, partition): one kernel per step instead
        (void)cudaGetLastError();
        return cudaSuccess;
    }
    e = note_err(c, e, "one-kernel CUDA-core pass");
    c->launches++;
    *launched = true;
    // the phases of the pass are not separate launches: the profile books the whole kernel under the heads
    prof_mark(c, 1, st);
    prof_mark(c, 2, st);
    prof_mark(c, 3, st);
    return e;
}

cudaError_t simt_draft(Ctx *c, const void *hidden, const float *logits0, const int32_t *row_index,
                       int M, int K, const mrp_draft_out &out, cudaStream_t st)
{
    if (M == 0) return cudaSuccess;
    if (fused_ok(c, M, K)) {
        bool launched = false;
        const cudaError_t e = c->cfg.dtype == MRP_F32
                                  ? simt_fused_t<float>(c, hidden, logits0, row_index, M, K, out, st, &launched)
                                  : simt_fused_t<__nv_bfloat16>(c, hidden, logits0, row_index, M, K, out, st, &launched);
        if (launched || e != cudaSuccess) return e;
    }
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
// (o16: the output as bf16 hi rows [n_rows, d] with the lo rows n_rows rows further on instead of fp32 rows in o)
__global__ void mod_attention_kernel(const float *__restrict__ q, const float *__restrict__ k,
                                     const float *__restrict__ v, int L, int d, int dh, float *__restrict__ o,
                                     __nv_bfloat16 *__restrict__ o16, int n_rows)
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
        if (L <= 64) {
            // blocks of up to 64 positions: lanes over the head's features (coalesced rows), one warp sum per key
            for (int j = 0; j < L; ++j) {
                const float *kj = k + ((size_t)b * L + j) * d + (size_t)hd * dh;
                float sdot = 0.f;
                for (int c = lane; c < dh; c += 32) sdot = fmaf(qi[c], kj[c], sdot);
                sdot = warp_sum(sdot) * scale;
                if (lane == 0) p[j] = sdot;
                mx = fmaxf(mx, sdot);
            }
        } else {
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
        }
        __syncwarp();
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
            const float val = acc / sum;
            const size_t at = ((size_t)b * L + i) * d + (size_t)hd * dh + c;
            if (o16) {
                const __nv_bfloat16 hh = __float2bfloat16_rn(val);
                o16[at] = hh;
                o16[(size_t)n_rows * d + at] = __float2bfloat16_rn(val - __bfloat162float(hh));
            } else {
                o[at] = val;
            }
        }
        __syncwarp();
    }
}

// The same behind a clean prefix (Fig. 1(c)): CTA = (block, attention head, chunk of the keys); keys and values are
// the first prefix_len[b] rows of the (sequence b, head) slab of the cache [*, H, cap, dh], then the block's own rows.  With `append`
// the block's keys and values are also stored behind the prefix rows (rows the call itself never reads).
template <typename T>
__global__ void __launch_bounds__(128) mod_attention_prefix_kernel(const float *__restrict__ q, const float *k, const float *v, int L,
                                                                   int d, int dh, int H, float *__restrict__ o,
                                                                   __nv_bfloat16 *__restrict__ o16, int n_rows, T *pk, T *pv,
                                                                   const int32_t *__restrict__ plen, int cap, int append, int n_ch,
                                                                   int gpc, int mma, float *part, int *counters,
                                                                   int32_t *__restrict__ status, int32_t *__restrict__ user_status)
{
    pdl_trigger();
    pdl_wait();
    extern __shared__ __align__(16) float att_sh[];
    const int unit = blockIdx.x, ch = unit % n_ch, bh = unit / n_ch, b = bh / H, hd = bh - b * H;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int P = plen[b];
    bool bad = P < 0 || P > cap;
    P = P < 0 ? 0 : (P > cap ? cap : P);
    const bool store = append && !bad && P + L <= cap;
    bad = bad || (append && !store);
    if (bad && threadIdx.x == 0 && hd == 0 && ch == 0) {
        atomicOr(status, MRP_DEV_BAD_INDEX);
        if (user_status) atomicOr(user_status, MRP_DEV_BAD_INDEX);
    }
    const size_t head = (size_t)hd * dh, slab = ((size_t)b * H + hd) * cap * dh, blk = (size_t)b * L * d + head;
    if (store && ch == 0) {
        for (int x = threadIdx.x; x < L * dh; x += 128) {
            const int i = x / dh, c = x - i * dh;
            pk[slab + (size_t)(P + i) * dh + c] = (T)k[blk + (size_t)i * d + c];
            pv[slab + (size_t)(P + i) * dh + c] = (T)v[blk + (size_t)i * d + c];
        }
    }
    att_unit<T, false>(q + blk, pk + slab, pv + slab, P, k + blk, v + blk, L, d, dh, ch, n_ch, gpc, mma,
                part + (size_t)bh * n_ch * L * (dh + 2), counters + bh, att_sh, warp, lane, [] { __syncthreads(); },
                [&](int i, int c, float val) {
                    const size_t at = blk + (size_t)i * d + c;
                    if (o16) {
                        const __nv_bfloat16 hh = __float2bfloat16_rn(val);
                        o16[at] = hh;
                        o16[(size_t)n_rows * d + at] = __float2bfloat16_rn(val - __bfloat162float(hh));
                    } else {
                        o[at] = val;
                    }
                });
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

// Rows every region of the module workspace is sized for: the positions of a call (max_seqs * block_len), rounded up
// to the row padding of the few-row tensor-core kernels where those may serve the call.
static size_t module_cap_rows(const mrp_config &cfg)
{
    const size_t cap = (size_t)cfg.max_seqs * cfg.block_len;
    return cap <= 128 ? (size_t)sk_head_pad((int)cap) : cap;
}

// ---- the module step as ONE kernel, for a handful of positions -----------------------------------
// With n = B * L <= 4 positions every matrix of the module is a matrix-vector product bound by its own weight
// stream (269 MB per step at d = 2048, F = 4096, D = 3), and a kernel per product leaves the stream idle
// between 33 launches.  Here the step is one cooperative kernel of 5 D + 2 phases between grid barriers (the
// barrier of the one-kernel drafting pass above):
//   [h ; emb[x]] -> z = W_proj .   | per layer: RMSNorm -> q, k, v | attention, a warp per (position, head)
//   | z += W_o o | RMSNorm -> silu(gate) * up | z += W_down a | h += z, LM-head operand of the masked rows.
// A product phase stages its input rows in shared memory (what other CTAs wrote: through L2) and every warp
// walks groups of four weight rows at once: each 16-byte read of an input row from shared memory then feeds four
// rows' products (one weight row at a time would need 128 bytes of shared memory per 16 bytes of weights), and
// four independent 16-byte weight loads are in flight per lane and iteration.  Where a product has fewer groups
// than the grid has warps its contraction is cut across the warps of a CTA, which add their parts in a fixed
// order.
constexpr int kModThreads = 512;
constexpr int kModRows = 4;            // positions (rows of every product)
constexpr int kModGroup = 4;           // weight rows a warp works on at a time
constexpr int kModMaxLayers = 8;
constexpr size_t kModMaxSmem = 200 * 1024;

template <typename T>
struct ModParams {
    const int32_t *tokens;
    const T *hidden0, *emb, *w_proj;
    float *h_state;
    const T *g_attn[kModMaxLayers], *w_q[kModMaxLayers], *w_k[kModMaxLayers], *w_v[kModMaxLayers], *w_o[kModMaxLayers];
    const T *g_mlp[kModMaxLayers], *w_gate[kModMaxLayers], *w_up[kModMaxLayers], *w_down[kModMaxLayers];
    int first_step, mask_token, emb_rows, n_layers;
    int n, B, L, d, F, H;
    float eps;
    float *z, *q, *k, *v, *act;            // module workspace, [n, d] each, act [n, F]
    const int32_t *row_index;
    int M;
    float *xt_f32;                         // LM-head operand rows h - h_0 of the masked rows: fp32 [M, d], or ...
    __nv_bfloat16 *xt_bf16;                // ... bf16 hi + lo rows behind the zero rows of step 0
    int lo_rows;
    __half *xt16;
    float *hidden_out;
    int32_t *status, *user_status;
    unsigned int *bar;
};

// Lane-partial products of kModGroup weight rows (nullptr: none), `len` columns each, with `rows` <= kModRows input
// rows in shared memory (fp32, row pitch `pitch`), then added over the lanes: every lane returns with all the
// sums.  bf16 rows of a multiple of 256 columns are read 16 bytes per lane.
template <typename T>
__device__ __forceinline__ void group_dots(const T *const (&wr)[kModGroup], const float *xs, int rows, int pitch, int len,
                                           int lane, float (&acc)[kModGroup][kModRows])
{
#pragma unroll
    for (int f = 0; f < kModGroup; ++f)
#pragma unroll
        for (int r = 0; r < kModRows; ++r) acc[f][r] = 0.f;
    if (std::is_same<T, __nv_bfloat16>::value && (len & 255) == 0) {
#pragma unroll 2
        for (int c = lane * 8; c < len; c += 256) {
            uint4 q[kModGroup];
#pragma unroll
            for (int f = 0; f < kModGroup; ++f)
                q[f] = wr[f] ? __ldg(reinterpret_cast<const uint4 *>(reinterpret_cast<const __nv_bfloat16 *>(wr[f]) + c))
                             : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
            for (int r = 0; r < kModRows; ++r) {
                if (r < rows) {
                    const float4 a = *reinterpret_cast<const float4 *>(xs + (size_t)r * pitch + c);
                    const float4 b = *reinterpret_cast<const float4 *>(xs + (size_t)r * pitch + c + 4);
#pragma unroll
                    for (int f = 0; f < kModGroup; ++f) {
                        float t = acc[f][r];
                        t = fmaf(__uint_as_float(q[f].x << 16), a.x, t); t = fmaf(__uint_as_float(q[f].x & 0xFFFF0000u), a.y, t);
                        t = fmaf(__uint_as_float(q[f].y << 16), a.z, t); t = fmaf(__uint_as_float(q[f].y & 0xFFFF0000u), a.w, t);
                        t = fmaf(__uint_as_float(q[f].z << 16), b.x, t); t = fmaf(__uint_as_float(q[f].z & 0xFFFF0000u), b.y, t);
                        t = fmaf(__uint_as_float(q[f].w << 16), b.z, t); t = fmaf(__uint_as_float(q[f].w & 0xFFFF0000u), b.w, t);
                        acc[f][r] = t;
                    }
                }
            }
        }
    } else {
#pragma unroll 4
        for (int c = lane; c < len; c += 32) {
            float wv[kModGroup];
#pragma unroll
            for (int f = 0; f < kModGroup; ++f) wv[f] = wr[f] ? ld_f(wr[f], c) : 0.f;
#pragma unroll
            for (int r = 0; r < kModRows; ++r) {
                if (r < rows) {
                    const float x = xs[(size_t)r * pitch + c];
#pragma unroll
                    for (int f = 0; f < kModGroup; ++f) acc[f][r] = fmaf(wv[f], x, acc[f][r]);
                }
            }
        }
    }
#pragma unroll
    for (int f = 0; f < kModGroup; ++f)
#pragma unroll
        for (int r = 0; r < kModRows; ++r) acc[f][r] = warp_sum(acc[f][r]);
}

// How the groups of a product are dealt out: the contraction is cut into S pieces (a power of two) when there
// are fewer groups than warps in the grid, so that all of them stream; the S warps of a group sit in one CTA
// and their partial sums are added there in a fixed order.
__device__ __forceinline__ int split_for(int n_groups, int n_in, int n_gw, bool wide)
{
    int S = 1;
    const int unit = wide ? 256 : 32;
    while (S < kModThreads / 32 && n_groups * (2 * S) <= n_gw && (n_in % (2 * S)) == 0 && ((n_in / (2 * S)) % unit) == 0) S *= 2;
    return S;
}

// One product of the step: y(g, f, r) for every group g of kModGroup weight rows (row(g, f): the row, or nullptr)
// and input row r, handed to epi(g, f, r, value) by one lane each.  xs: the input rows in shared memory (pitch
// n_in); red: kModThreads / 32 * 16 floats of shared memory.  Every thread of the CTA calls it.
template <typename T, typename RowFn, typename Epi>
__device__ __forceinline__ void gemv_phase(RowFn row, Epi epi, const float *xs, int rows, int n_in, int n_groups, int S,
                                           float *red)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = kModThreads / 32;
    const int G = gridDim.x, cta = blockIdx.x;
    const int per_round = n_warps / S, team = warp / S, split = warp % S, chunk = n_in / S;
    const int rounds = (n_groups + G * per_round - 1) / (G * per_round);
    for (int rd = 0; rd < rounds; ++rd) {
        const int g = (rd * G + cta) * per_round + team;
        const T *wr[kModGroup];
        float acc[kModGroup][kModRows];
#pragma unroll
        for (int f = 0; f < kModGroup; ++f) {
            const T *w = g < n_groups ? row(g, f) : nullptr;
            wr[f] = w ? w + (size_t)split * chunk : nullptr;
        }
        group_dots<T>(wr, xs + (size_t)split * chunk, rows, n_in, chunk, lane, acc);
        // lane f * kModRows + r takes sum (f, r)
        float mine = 0.f;
#pragma unroll
        for (int f = 0; f < kModGroup; ++f)
#pragma unroll
            for (int r = 0; r < kModRows; ++r)
                if (lane == f * kModRows + r) mine = acc[f][r];
        if (S > 1) {
            if (lane < kModGroup * kModRows) red[warp * 16 + lane] = mine;
            __syncthreads();
            if (split == 0 && lane < kModGroup * kModRows) {
                mine = red[warp * 16 + lane];
                for (int s2 = 1; s2 < S; ++s2) mine += red[(warp + s2) * 16 + lane];
            }
        }
        if (split == 0 && lane < kModGroup * kModRows && g < n_groups) epi(g, lane / kModRows, lane % kModRows, mine);
        if (S > 1) __syncthreads();
    }
}

// Rows [n, width] of a buffer another phase wrote, into shared memory (through L2).
__device__ __forceinline__ void stage_rows(float *dst, const float *src, int count)
{
    if ((count & 3) == 0) {
#pragma unroll 8
        for (int i = threadIdx.x * 4; i < count; i += blockDim.x * 4)
            *reinterpret_cast<float4 *>(dst + i) = __ldcg(reinterpret_cast<const float4 *>(src + i));
    } else {
        for (int i = threadIdx.x; i < count; i += blockDim.x) dst[i] = __ldcg(src + i);
    }
}

// RMSNorm of the n rows in shared memory, in place (warp per row).
template <typename T>
__device__ __forceinline__ void norm_rows(float *xs, int n, int d, const T *gamma, float eps)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int r = warp; r < n; r += (int)(blockDim.x >> 5)) {
        float ss = 0.f;
        for (int j = lane; j < d; j += 32) ss = fmaf(xs[(size_t)r * d + j], xs[(size_t)r * d + j], ss);
        ss = warp_sum(ss);
        const float rstd = rsqrtf(ss / (float)d + eps);
        for (int j = lane; j < d; j += 32) xs[(size_t)r * d + j] = xs[(size_t)r * d + j] * rstd * ld_f(gamma, j);
    }
}

template <typename T>
__global__ void __launch_bounds__(kModThreads)
module_fused_kernel(const ModParams<T> p)
{
    extern __shared__ __align__(16) float sh[];
    __shared__ float red[kModThreads / 32 * 16];
    __shared__ int inv[kModRows];            // dense position -> masked row, or -1
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_warps = kModThreads / 32;
    const int G = gridDim.x, cta = blockIdx.x;
    const int gw = cta * n_warps + warp, n_gw = G * n_warps;
    const int n = p.n, d = p.d, F = p.F, L = p.L;
    const bool wide = std::is_same<T, __nv_bfloat16>::value;
    FusedSync sy;
    sy.base = *reinterpret_cast<volatile unsigned int *>(p.bar + 1);
    sy.done = 0;
    sy.total = 5 * p.n_layers + 2;
    auto leave = [&]() {
        if (cta == 0 && threadIdx.x == 0) {
            *reinterpret_cast<volatile unsigned int *>(p.bar + 1) = sy.base + (unsigned int)sy.total * G;
            __threadfence();
        }
    };
    // the products of the step: groups of kModGroup weight rows and how their contraction is split
    const int ng_d = (d + kModGroup - 1) / kModGroup, ng_qkv = 3 * d / kModGroup, ng_gu = (F + 1) / 2;
    const int s_proj = split_for(ng_d, 2 * d, n_gw, wide), s_qkv = split_for(ng_qkv, d, n_gw, wide);
    const int s_o = split_for(ng_d, d, n_gw, wide), s_gu = split_for(ng_gu, d, n_gw, wide), s_dn = split_for(ng_d, F, n_gw, wide);
    auto row_proj = [&](int g, int f) { const int j = g * kModGroup + f; return j < d ? p.w_proj + (size_t)j * 2 * d : (const T *)nullptr; };
    auto rows_of = [&](const T *w, int n_in) {
        return [=](int g, int f) { const int j = g * kModGroup + f; return j < d ? w + (size_t)j * n_in : (const T *)nullptr; };
    };
    auto row_qkv = [&](int l) {
        const T *wq = p.w_q[l], *wk = p.w_k[l], *wv = p.w_v[l];
        return [=](int g, int f) {                      // (kModGroup divides d: a group stays within one matrix)
            const int j = g * kModGroup + f, which = j / d;
            return (which == 0 ? wq : which == 1 ? wk : wv) + (size_t)(j - which * d) * d;
        };
    };
    auto row_gu = [&](int l) {
        const T *wg = p.w_gate[l], *wu = p.w_up[l];
        return [=](int g, int f) {                      // rows 0, 1: gate and up of feature 2 g; rows 2, 3: of feature 2 g + 1
            const int ft = 2 * g + (f >> 1);
            return ft < F ? ((f & 1) ? wu : wg) + (size_t)ft * d : (const T *)nullptr;
        };
    };
    auto add_to_z = [&](int g, int f, int r, float v) {
        const int j = g * kModGroup + f;
        if (j < d && r < n) { float *dst = p.z + (size_t)r * d + j; *dst = __ldcg(dst) + v; }
    };

    // ---- z = W_proj [h ; emb[x]] ----
    for (int i = 0; i < n; ++i) {
        int tok = p.tokens[i];
        if (tok >= p.emb_rows || tok < -1) {          // outside the table: reads as masked, raises the bit
            if (cta == 0 && threadIdx.x == 0) {
                atomicOr(p.status, MRP_DEV_BAD_INDEX);
                if (p.user_status) atomicOr(p.user_status, MRP_DEV_BAD_INDEX);
            }
            tok = -1;
        }
        if (tok < 0) tok = p.mask_token;
        for (int j = threadIdx.x; j < d; j += blockDim.x) {
            const float h = p.first_step ? ld_f(p.hidden0, (size_t)i * d + j) : __ldcg(p.h_state + (size_t)i * d + j);
            if (p.first_step && i % G == cta) p.h_state[(size_t)i * d + j] = h;
            sh[(size_t)i * 2 * d + j] = h;
            sh[(size_t)i * 2 * d + d + j] = ld_f(p.emb, (size_t)tok * d + j);
        }
    }
    __syncthreads();
    gemv_phase<T>(row_proj, [&](int g, int f, int r, float v) {
        const int j = g * kModGroup + f;
        if (j < d && r < n) p.z[(size_t)r * d + j] = v;
    }, sh, n, 2 * d, ng_d, s_proj, red);
    if (!fused_barrier(p, sy)) { leave(); return; }

    for (int l = 0; l < p.n_layers; ++l) {
        // ---- q, k, v of RMSNorm(z) g_attn: one product over 3 d output features ----
        stage_rows(sh, p.z, n * d);
        __syncthreads();
        norm_rows<T>(sh, n, d, p.g_attn[l], p.eps);
        __syncthreads();
        gemv_phase<T>(row_qkv(l), [&](int g, int f, int r, float v) {
            const int j = g * kModGroup + f, which = j / d;
            if (r < n) (which == 0 ? p.q : which == 1 ? p.k : p.v)[(size_t)r * d + (j - which * d)] = v;
        }, sh, n, d, ng_qkv, s_qkv, red);
        if (!fused_barrier(p, sy)) { leave(); return; }

        // ---- block-local bidirectional attention: a warp per (position, attention head) ----
        {
            const int dh = d / p.H;
            const float scale = rsqrtf((float)dh);
            for (int item = gw; item < n * p.H; item += n_gw) {
                const int i = item / p.H, hd = item - i * p.H, b = i / L;
                const float *qi = p.q + (size_t)i * d + (size_t)hd * dh;
                float sc[kModRows], mx = -INFINITY;
#pragma unroll
                for (int j = 0; j < kModRows; ++j) {
                    sc[j] = -INFINITY;
                    if (j < L) {
                        const float *kj = p.k + ((size_t)b * L + j) * d + (size_t)hd * dh;
                        float t = 0.f;
                        for (int c = lane; c < dh; c += 32) t = fmaf(__ldcg(qi + c), __ldcg(kj + c), t);
                        sc[j] = warp_sum(t) * scale;
                        mx = fmaxf(mx, sc[j]);
                    }
                }
                float sum = 0.f;
#pragma unroll
                for (int j = 0; j < kModRows; ++j) {
                    sc[j] = j < L ? expf(sc[j] - mx) : 0.f;
                    sum += sc[j];
                }
                for (int c = lane; c < dh; c += 32) {
                    float a = 0.f;
#pragma unroll
                    for (int j = 0; j < kModRows; ++j)
                        if (j < L) a = fmaf(sc[j], __ldcg(p.v + ((size_t)b * L + j) * d + (size_t)hd * dh + c), a);
                    p.act[(size_t)i * d + (size_t)hd * dh + c] = a / sum;       // (the activation buffer is free here)
                }
            }
        }
        if (!fused_barrier(p, sy)) { leave(); return; }

        // ---- z += W_o o ----
        stage_rows(sh, p.act, n * d);
        __syncthreads();
        gemv_phase<T>(rows_of(p.w_o[l], d), add_to_z, sh, n, d, ng_d, s_o, red);
        if (!fused_barrier(p, sy)) { leave(); return; }

        // ---- a = silu(W_gate n) * (W_up n), n = RMSNorm(z) g_mlp: two features (four weight rows) per group ----
        stage_rows(sh, p.z, n * d);
        __syncthreads();
        norm_rows<T>(sh, n, d, p.g_mlp[l], p.eps);
        __syncthreads();
        {
            // gate and up of a feature land in neighbouring lanes: lane f * kModRows + r holds row f of the group
            gemv_phase<T>(row_gu(l), [&](int g, int f, int r, float v) {
                // (every lane below 16 is here together: the up sum sits kModRows lanes above the gate sum)
                const float us = __shfl_down_sync(0x0000ffffu, v, kModRows);
                const int ft = 2 * g + (f >> 1);
                if (!(f & 1) && ft < F && r < n) p.act[(size_t)r * F + ft] = v / (1.f + expf(-v)) * us;
            }, sh, n, d, ng_gu, s_gu, red);
        }
        if (!fused_barrier(p, sy)) { leave(); return; }

        // ---- z += W_down a ----
        stage_rows(sh, p.act, n * F);
        __syncthreads();
        gemv_phase<T>(rows_of(p.w_down[l], F), add_to_z, sh, n, F, ng_d, s_dn, red);
        if (!fused_barrier(p, sy)) { leave(); return; }
    }

    // ---- h <- h + Delta at every position; the LM-head operand h - h_0 of the masked rows ----
    if (threadIdx.x < kModRows) inv[threadIdx.x] = -1;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int m = 0; m < p.M; ++m) {
            const int idx = p.row_index ? p.row_index[m] : m;
            if (row_ok(idx, n)) inv[idx] = m;
            else if (cta == 0) {
                atomicOr(p.status, MRP_DEV_BAD_INDEX);
                if (p.user_status) atomicOr(p.user_status, MRP_DEV_BAD_INDEX);
            }
        }
    }
    __syncthreads();
    auto put_operand = [&](int m, int j, float h, float r) {
        if (p.hidden_out) p.hidden_out[(size_t)m * d + j] = h;
        if (p.xt_f32) p.xt_f32[(size_t)m * d + j] = r;
        if (p.xt_bf16) {
            const __nv_bfloat16 hi = __float2bfloat16_rn(r);
            p.xt_bf16[(size_t)m * d + j] = __float2bfloat16(0.f);                          // step 0 has no residual
            p.xt_bf16[((size_t)p.lo_rows + m) * d + j] = __float2bfloat16(0.f);
            p.xt_bf16[((size_t)p.M + m) * d + j] = hi;
            p.xt_bf16[((size_t)p.lo_rows + p.M + m) * d + j] = __float2bfloat16_rn(r - __bfloat162float(hi));
            if (p.xt16) p.xt16[(size_t)m * d + j] = __float2half_rn(r);
        }
    };
    for (int e = cta * kModThreads + threadIdx.x; e < n * d; e += G * kModThreads) {
        const int i = e / d, j = e - i * d;
        const float h = __ldcg(p.h_state + e) + __ldcg(p.z + e);
        p.h_state[e] = h;
        if (inv[i] >= 0) put_operand(inv[i], j, h, h - ld_f(p.hidden0, (size_t)e));
    }
    // rows whose index was out of range read as zeros
    for (int m = 0; m < p.M; ++m) {
        const int idx = p.row_index ? p.row_index[m] : m;
        if (!row_ok(idx, n) || inv[idx] != m)
            for (int j = cta * kModThreads + threadIdx.x; j < d; j += G * kModThreads) put_operand(m, j, 0.f, 0.f);
    }
    fused_barrier(p, sy);
    leave();
}

static size_t module_fused_smem(int n, int d, int F)
{
    size_t fl = (size_t)n * 2 * d;
    if ((size_t)n * F > fl) fl = (size_t)n * F;
    return fl * 4;
}

// Launches the one-kernel module step if the shape fits it (*launched tells).
template <typename T>
static cudaError_t module_fused_t(Ctx *c, const int32_t *tokens, const void *hidden0, float *h_state, const int32_t *row_index,
                                  int M, int B, int L, bool first_step, const mrp_draft_out &out, cudaStream_t st,
                                  float *xt_f32, __nv_bfloat16 *xt_bf16, int lo_rows, __half *xt16, bool *launched)
{
    *launched = false;
    const mrp_module_weights &w = c->module;
    const int d = c->cfg.d, F = c->cfg.d_ff, n = B * L;
    // (with a clean prefix attached the attention runs in the per-product form or in the tensor-core step)
    if (c->has_prefix || n > kModRows || L > kModRows || w.n_layers > kModMaxLayers || (c->cfg.flags & MRP_FLAG_NO_CHAIN) || (d & 3) || (F & 3) || F < d ||
        module_fused_smem(n, d, F) > kModMaxSmem)
        return cudaSuccess;
    auto kern = module_fused_kernel<T>;
    static std::atomic<unsigned long long> asked{0}, fits{0};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const unsigned long long bit = 1ull << (dev & 63);
    if (!(asked.load() & bit)) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kModMaxSmem);
        if (e != cudaSuccess) return e;
        int per_sm = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kModThreads, kModMaxSmem);
        if (e != cudaSuccess) return e;
        if (per_sm >= 1) fits.fetch_or(bit);
        asked.fetch_or(bit);
    }
    if (!(fits.load() & bit)) return cudaSuccess;
    ModParams<T> p;
    memset(&p, 0, sizeof(p));
    p.tokens = tokens; p.hidden0 = (const T *)hidden0; p.emb = (const T *)w.emb; p.w_proj = (const T *)w.w_proj;
    p.h_state = h_state;
    for (int l = 0; l < w.n_layers; ++l) {
        const mrp_module_layer &y = w.layers[l];
        p.g_attn[l] = (const T *)y.g_attn; p.w_q[l] = (const T *)y.w_q; p.w_k[l] = (const T *)y.w_k; p.w_v[l] = (const T *)y.w_v;
        p.w_o[l] = (const T *)y.w_o; p.g_mlp[l] = (const T *)y.g_mlp; p.w_gate[l] = (const T *)y.w_gate;
        p.w_up[l] = (const T *)y.w_up; p.w_down[l] = (const T *)y.w_down;
    }
    p.first_step = first_step ? 1 : 0; p.mask_token = w.mask_token; p.emb_rows = w.emb_rows; p.n_layers = w.n_layers;
    p.n = n; p.B = B; p.L = L; p.d = d; p.F = F; p.H = w.n_attn_heads; p.eps = c->cfg.rms_eps;
    const size_t cap = module_cap_rows(c->cfg);
    char *ws = c->module_ws;
    auto take = [&](size_t bytes) { char *p0 = ws; ws += align_up(bytes, 256); return (float *)p0; };
    take(cap * 2 * d * 4);                 // (the concatenated rows of the separate kernels)
    p.z = take(cap * d * 4);
    take(cap * d * 4);
    p.q = take(cap * d * 4); p.k = take(cap * d * 4); p.v = take(cap * d * 4);
    take(cap * d * 4);
    p.act = take(cap * F * 4);
    p.row_index = row_index; p.M = M;
    p.xt_f32 = xt_f32; p.xt_bf16 = xt_bf16; p.lo_rows = lo_rows; p.xt16 = xt16; p.hidden_out = out.hidden_out;
    p.status = (int32_t *)(c->ws + c->lay.status); p.user_status = out.status;
    p.bar = (unsigned int *)(c->ws + c->lay.status) + 16;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(c->sm_count);
    cfg.blockDim = dim3(kModThreads);
    cfg.dynamicSmemBytes = module_fused_smem(n, d, F);
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeCooperative;
    at[0].val.cooperative = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, kern, p);
    if (e == cudaErrorCooperativeLaunchTooLarge) {
        // the context may use fewer SMs than the device has (MPS share, partition): one kernel per product instead
        (void)cudaGetLastError();
        return cudaSuccess;
    }
    e = note_err(c, e, "one-kernel module step");
    c->launches++;
    *launched = true;
    return e;
}

// ---- the module's products on the tensor cores (more than a handful of positions) ----------------------
// The matrix products of the step run on the row-major tcgen05 kernel (tc_linear / tc_gate_up: bf16 hi + lo
// operand rows, fp32 accumulation, RMSNorm folded in as gamma on the operand and 1 / rms on the result; a product
// that completes z writes the next product's operand and its partial sums of squares itself); the embedding
// fusion in front and the attention stay on the CUDA cores.
// bf16 hi + lo rows of [h_i ; emb[x_i]]: the hi rows [n, 2 d], the lo rows lo_rows rows further on.
__global__ void mod_cat_split_kernel(const float *h_state, const __nv_bfloat16 *__restrict__ hidden0, int first_step,
                                     const int32_t *__restrict__ tokens, const __nv_bfloat16 *__restrict__ emb, int mask_token,
                                     int emb_rows, int lo_rows, int d, float *h_out /* = h_state */, __nv_bfloat16 *__restrict__ cat,
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
    __nv_bfloat16 *hi = cat + (size_t)i * 2 * d, *lo = cat + ((size_t)lo_rows + i) * 2 * d;
    for (int j = threadIdx.x; j < d; j += blockDim.x) {
        const float h = first_step ? __bfloat162float(hidden0[(size_t)i * d + j]) : h_state[(size_t)i * d + j];
        if (first_step) h_out[(size_t)i * d + j] = h;
        const __nv_bfloat16 hh = __float2bfloat16_rn(h);
        hi[j] = hh;
        lo[j] = __float2bfloat16_rn(h - __bfloat162float(hh));
        hi[d + j] = emb[(size_t)tok * d + j];            // a bf16 value: no remainder
        lo[d + j] = __float2bfloat16(0.f);
    }
}

// Whether the module's products of a call over n positions can run on the tensor cores.
static bool module_tc_ok(const Ctx *c, int n)
{
    if (!c->use_tc || c->cfg.dtype != MRP_BF16 || (c->cfg.flags & MRP_FLAG_FORCE_SIMT)) return false;
    // (the partial sums of squares of the module's norms use the context's [kSumsqSlices, max_rows] array)
    if (c->cfg.d % 64 || c->cfg.d_ff % 64 || (long long)c->sm_count * n > (long long)c->cfg.max_rows * kSumsqSlices) return false;
    const mrp_module_weights &w = c->module;
    auto al = [](const void *p) { return ((uintptr_t)p & 15u) == 0; };
    if (!al(w.emb) || !al(w.w_proj)) return false;
    for (int l = 0; l < w.n_layers; ++l) {
        const mrp_module_layer &y = w.layers[l];
        if (!al(y.w_q) || !al(y.w_k) || !al(y.w_v) || !al(y.w_o) || !al(y.w_gate) || !al(y.w_up) || !al(y.w_down)) return false;
    }
    return true;
}

// Whether a call over n positions runs as one cooperative tensor-core kernel.
static bool module_chain_ok(Ctx *c, int n, int L, cudaStream_t st)
{
    const mrp_module_weights &w = c->module;
    return module_tc_ok(c, n) && w.n_layers > 0 && n <= 64 && (size_t)sk_head_pad(n) <= module_cap_rows(c->cfg) &&
           sk_heads_ok(c->cfg) && !(c->cfg.flags & (MRP_FLAG_ROW_MAJOR_ONLY | MRP_FLAG_NO_CHAIN)) &&
           sk_module_step(c, n, L, nullptr, nullptr, nullptr, false, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr,
                          nullptr, nullptr, nullptr, 0, 0, false, nullptr, nullptr, st, true) == cudaSuccess;
}

// The attention of layer l over B blocks of L positions: block-local, or behind the context's clean prefix.
template <typename T>
static cudaError_t module_attention(Ctx *c, int layer, int B, int L, const float *q, const float *k, const float *v, float *o,
                                    __nv_bfloat16 *o16, int n_rows, const mrp_draft_out &out, cudaStream_t st)
{
    const mrp_module_weights &w = c->module;
    const int d = c->cfg.d, dh = d / w.n_attn_heads;
    const bool pdl = !(c->cfg.flags & MRP_FLAG_NO_PDL);
    c->launches++;
    if (!c->has_prefix)
        return launch_k(mod_attention_kernel, dim3(B, w.n_attn_heads), dim3(128), (size_t)4 * L * 4, st, pdl, q, k, v, L, d, dh, o, o16,
                        n_rows);
    // the keys of a (block, head) split over CTAs where there are few of those; the partial results and the arrival
    // counters (zero before and after every launch) sit behind the module's other workspace
    // (this kernel keeps the CUDA-core routine: with three CTAs per SM it is as fast here as the tensor-core routine of
    // the one-kernel step, which takes 248 registers)
    const bool mma = false;
    const AttSplit sp = att_split(c->prefix_cap, L, B * w.n_attn_heads, dh, 8 * c->sm_count);
    float *part = (float *)(c->module_ws + module_att_offset(c->cfg));
    int *counters = (int *)(part + kAttPartFloats);
    return launch_k(mod_attention_prefix_kernel<T>, dim3((unsigned)(B * w.n_attn_heads * sp.n_ch)), dim3(128),
                    (size_t)att_sh_floats(dh) * 4, st, pdl, q, k, v, L, d, dh, w.n_attn_heads, o, o16, n_rows,
                    (T *)c->prefix_layers[layer].k, (T *)c->prefix_layers[layer].v, c->prefix_len, c->prefix_cap,
                    c->prefix_append ? 1 : 0, sp.n_ch, sp.gpc, mma ? 1 : 0, part, counters, (int32_t *)(c->ws + c->lay.status),
                    out.status);
}

// The module itself (everything in front of `h <- h + Delta`) with its products on the tensor cores.
static cudaError_t module_body_tc(Ctx *c, const int32_t *tokens, const void *hidden0, float *h_state, int B, int L,
                                  bool first_step, const mrp_draft_out &out, cudaStream_t st, float *z)
{
    const mrp_module_weights &w = c->module;
    const int d = c->cfg.d, F = c->cfg.d_ff, n = B * L, dh = d / w.n_attn_heads;
    const size_t cap = module_cap_rows(c->cfg);
    char *ws = c->module_ws;
    auto take = [&](size_t bytes) { char *p0 = ws; ws += align_up(bytes, 256); return p0; };
    // the regions of the fp32 path hold the bf16 hi + lo operands here (same bytes: two halves of two bytes)
    __nv_bfloat16 *cat16 = (__nv_bfloat16 *)take(cap * 2 * d * 4);
    float *zz = (float *)take(cap * d * 4);
    __nv_bfloat16 *xa = (__nv_bfloat16 *)take(cap * d * 4);          // operand of q/k/v and of gate/up
    float *q = (float *)take(cap * d * 4), *k = (float *)take(cap * d * 4), *v = (float *)take(cap * d * 4);
    __nv_bfloat16 *xb = (__nv_bfloat16 *)take(cap * d * 4);          // operand of the output projection
    __nv_bfloat16 *act16 = (__nv_bfloat16 *)take(cap * F * 4);
    (void)zz;
    float *sumsq = (float *)(c->ws + c->lay.sumsq);
    int32_t *status = (int32_t *)(c->ws + c->lay.status);
    const bool pdl = !(c->cfg.flags & MRP_FLAG_NO_PDL);
    // where the lo rows of an operand sit behind its hi rows: the few-row kernels fetch both with one TMA box
    const bool few = sk_head_rows_ok(n) && sk_heads_ok(c->cfg) && (size_t)sk_head_pad(n) <= cap &&
                     !(c->cfg.flags & MRP_FLAG_ROW_MAJOR_ONLY);
    const int lo_rows = few ? sk_head_pad(n) : n;
    cudaError_t e = launch_k(mod_cat_split_kernel, dim3(n), dim3(256), 0, st, pdl, (const float *)h_state,
                             (const __nv_bfloat16 *)hidden0, first_step ? 1 : 0, tokens, (const __nv_bfloat16 *)w.emb, w.mask_token,
                             w.emb_rows, lo_rows, d, h_state, cat16, status, out.status);
    c->launches++;
    // Every product that completes z also writes the next product's operand (z * next norm weight, hi + lo) and
    // its partial sums of squares: no kernel between them.
    int n_ss = 1;
    const void *g_first = w.n_layers > 0 ? w.layers[0].g_attn : nullptr;
    if (few) {
        // up to 64 positions: the few-row kernels (weight rows on the MMA M axis, contraction split over CTAs), whose
        // tiles stream the weights once whatever the number of positions.  Their per-tile arrival counters must be
        // zero at the first launch (every launch leaves them at zero again).
        if (e == cudaSuccess) e = cudaMemsetAsync(c->ws + c->lay.sk_counters, 0, (size_t)kSkMaxTiles * 4, st);
        if (e == cudaSuccess)
            e = sk_linear(c, cat16, n, 2 * d, w.w_proj, d, nullptr, 1, z, false, g_first, g_first ? xa : nullptr, sumsq, &n_ss,
                          out.status, st);
        for (int l = 0; l < w.n_layers && e == cudaSuccess; ++l) {
            const mrp_module_layer &y = w.layers[l];
            e = sk_linear3(c, xa, n, d, y.w_q, y.w_k, y.w_v, d, sumsq, n_ss, q, k, v, out.status, st);
            if (e == cudaSuccess) e = module_attention<__nv_bfloat16>(c, l, B, L, q, k, v, nullptr, xb, lo_rows, out, st);
            if (e == cudaSuccess)
                e = sk_linear(c, xb, n, d, y.w_o, d, nullptr, 1, z, true, y.g_mlp, xa, sumsq, &n_ss, out.status, st);
            if (e == cudaSuccess) e = sk_gate_up(c, xa, n, d, y.w_gate, y.w_up, F, sumsq, n_ss, act16, out.status, st);
            const void *g_next = l + 1 < w.n_layers ? w.layers[l + 1].g_attn : nullptr;
            if (e == cudaSuccess)
                e = sk_linear(c, act16, n, F, y.w_down, d, nullptr, 1, z, true, g_next, g_next ? xa : nullptr, sumsq, &n_ss,
                              out.status, st);
        }
        return e;
    }
    if (e == cudaSuccess)
        e = tc_linear(c, cat16, n, 2 * d, w.w_proj, d, nullptr, 1, z, false, out.status, st, g_first, g_first ? xa : nullptr,
                      sumsq, &n_ss);
    for (int l = 0; l < w.n_layers && e == cudaSuccess; ++l) {
        const mrp_module_layer &y = w.layers[l];
        e = tc_linear3(c, xa, n, d, y.w_q, y.w_k, y.w_v, d, sumsq, n_ss, q, k, v, out.status, st);
        if (e == cudaSuccess) e = module_attention<__nv_bfloat16>(c, l, B, L, q, k, v, nullptr, xb, n, out, st);
        if (e == cudaSuccess)
            e = tc_linear(c, xb, n, d, y.w_o, d, nullptr, 1, z, true, out.status, st, y.g_mlp, xa, sumsq, &n_ss);
        if (e == cudaSuccess) e = tc_gate_up(c, xa, n, d, y.w_gate, y.w_up, F, sumsq, n_ss, act16, out.status, st);
        const void *g_next = l + 1 < w.n_layers ? w.layers[l + 1].g_attn : nullptr;
        if (e == cudaSuccess)
            e = tc_linear(c, act16, n, F, y.w_down, d, nullptr, 1, z, true, out.status, st, g_next, g_next ? xa : nullptr, sumsq,
                          &n_ss);
    }
    return e;
}

// Where the clean-prefix attention's area starts: the partial results of split units, then their arrival counters
// (zeroed at the start of every step that uses them).
size_t module_att_offset(const mrp_config &cfg)
{
    const size_t n = module_cap_rows(cfg), d = (size_t)cfg.d, F = (size_t)cfg.d_ff;
    // (the last term: the arrival counters of the one-launch tensor-core step)
    return align_up(n * 2 * d * 4, 256) + 6 * align_up(n * d * 4, 256) + align_up(n * F * 4, 256) +
           align_up((size_t)kModChainBarInts * 4, 256);
}

size_t module_workspace_bytes(const mrp_config &cfg, int n_layers)
{
    (void)n_layers;
    return module_att_offset(cfg) + align_up(kAttPartFloats * 4, 256) + align_up((size_t)kAttCounters * 4, 256);
}

template <typename T>
static cudaError_t module_step_t(Ctx *c, const int32_t *tokens, const void *hidden0, float *h_state, const float *logits0,
                                 const int32_t *row_index, int M, int B, int L, bool first_step, const mrp_draft_out &out,
                                 cudaStream_t st)
{
    const mrp_module_weights &w = c->module;
    const int d = c->cfg.d, F = c->cfg.d_ff, n = B * L, dh = d / w.n_attn_heads;
    const size_t cap = module_cap_rows(c->cfg);
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
    float *att_part = (float *)(c->module_ws + module_att_offset(c->cfg));
    if (c->has_prefix) {
        // the arrival counters of the clean-prefix attention's split units start at zero (every launch leaves them so)
        const cudaError_t ez = cudaMemsetAsync(att_part + kAttPartFloats, 0, (size_t)kAttCounters * 4, st);
        if (ez != cudaSuccess) return ez;
    }
    if (module_chain_ok(c, n, L, st)) {
        // up to 64 positions on a tensor-core context: the whole step (fusion, the layers, h <- h + Delta, the LM-head
        // operand) as one cooperative tcgen05 kernel, then the LM-head kernels.  (At four positions, decode shape:
        // 0.14 ms against 0.225 ms for the one CUDA-core kernel below, which serves the contexts and shapes this
        // one does not.)
        TcPlan pl;
        if (M > 0) pl = tc_plan(c, M, 1, out, st, false);
        char *wp = c->module_ws;
        auto tk = [&](size_t bytes) { char *p0 = wp; wp += align_up(bytes, 256); return p0; };
        __nv_bfloat16 *cat16 = (__nv_bfloat16 *)tk(cap * 2 * d * 4);
        float *zc = (float *)tk(cap * d * 4);
        __nv_bfloat16 *xa = (__nv_bfloat16 *)tk(cap * d * 4);
        float *qc = (float *)tk(cap * d * 4), *kc2 = (float *)tk(cap * d * 4), *vc = (float *)tk(cap * d * 4);
        __nv_bfloat16 *xb = (__nv_bfloat16 *)tk(cap * d * 4);
        __nv_bfloat16 *act16 = (__nv_bfloat16 *)tk(cap * F * 4);
        int32_t *bar_mem = (int32_t *)wp;
        const cudaError_t ec = sk_module_step(c, n, L, tokens, hidden0, h_state, first_step, cat16, xa, xb, act16, qc, kc2, vc, zc,
                                              bar_mem, row_index, M, c->lo_xt, M > 0 && pl.f16_lm, out.hidden_out, out.status, st,
                                              false, att_part, (int *)(att_part + kAttPartFloats));
        if (ec != cudaSuccess || M == 0) return ec;
        return tc_lm_tail(c, pl, logits0, row_index, M, 1, out, st);
    } else {
        // a handful of positions: the whole module step as one kernel, then the LM-head kernels
        bool launched = false;
        TcPlan pl;
        if (c->use_tc && M > 0) pl = tc_plan(c, M, 1, out, st, false);
        __nv_bfloat16 *xtb = c->use_tc ? (__nv_bfloat16 *)(c->ws + c->lay.xt) : nullptr;
        const cudaError_t ef = module_fused_t<T>(c, tokens, hidden0, h_state, row_index, M, B, L, first_step, out, st,
                                                 c->use_tc ? (float *)nullptr : (float *)(c->ws + c->lay.xt), xtb, c->lo_xt,
                                                 (c->use_tc && M > 0 && pl.f16_lm) ? (__half *)(c->ws + c->lay.xt16) : (__half *)nullptr,
                                                 &launched);
        if (ef != cudaSuccess) return ef;
        if (launched) {
            if (M == 0) return cudaSuccess;
            return c->use_tc ? tc_lm_tail(c, pl, logits0, row_index, M, 1, out, st) : simt_lm_tail(c, logits0, row_index, M, 1, out, st);
        }
    }
    const bool on_tc = module_tc_ok(c, n);
    cudaError_t e = cudaSuccess;
    if (on_tc) {
        e = module_body_tc(c, tokens, hidden0, h_state, B, L, first_step, out, st, z);
    } else {
        e = launch_k(mod_concat_kernel<T>, dim3(n), dim3(256), 0, st, pdl, (const float *)h_state, (const T *)hidden0,
                     first_step ? 1 : 0, tokens, (const T *)w.emb, w.mask_token, w.emb_rows, d, h_state, cat, status, out.status);
        c->launches++;
        if (e == cudaSuccess) e = lin(w.w_proj, cat, 2 * d, d, z, 0);
    }
    for (int l = 0; l < (on_tc ? 0 : w.n_layers) && e == cudaSuccess; ++l) {
        const mrp_module_layer &y = w.layers[l];
        e = launch_k(rmsnorm_kernel<T>, dim3(n), dim3(256), 0, st, pdl, (const float *)z, (const T *)y.g_attn, d, c->cfg.rms_eps, nn);
        c->launches++;
        if (e == cudaSuccess) e = lin(y.w_q, nn, d, d, q, 0);
        if (e == cudaSuccess) e = lin(y.w_k, nn, d, d, k, 0);
        if (e == cudaSuccess) e = lin(y.w_v, nn, d, d, v, 0);
        if (e == cudaSuccess) e = module_attention<T>(c, l, B, L, q, k, v, o, nullptr, n, out, st);
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
