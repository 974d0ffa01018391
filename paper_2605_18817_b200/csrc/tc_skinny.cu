// Tensor-core kernels for few activation rows (sm_100a): the weight rows sit on the MMA M axis
// (128 TMEM lanes, one weight row per epilogue thread) and the activation rows on the N axis,
// so a k-chunk of a stage is 16 KB of weights next to a few KB of activations and the ring of
// TMA stages holds almost nothing but weight bytes in flight.  Same three GEMMs, same operand
// buffers and same results as the row-major family (tc_kernels.cu):
//   GU  gate/up + SwiGLU (a tile = 64 gate rows on lanes 0-63, their 64 up rows on 64-127)
//   DN  down projection, h <- h + Delta, operands of the next GEMMs, partial sums of squares
//   LM  shared LM head on the stacked rows h_k - h_0, "+ l_0", online softmax statistics kept
//       per (thread, row-step) in registers and merged once per CTA                  (a2, a3)
// Each activation operand is a bf16 hi block followed by a bf16 lo block; a stage holds both as
// one B tile of N = 2 * RP rows, so one MMA per k-step yields the products with hi in columns
// [0, RP) and with lo in [RP, 2 RP) of the accumulator; the epilogue adds the two.
// LM: every CTA owns a contiguous range of 16-row vocabulary units, cut into the fewest tiles of
// at most 128 rows, all (nearly) equally high; each height has its own tensor map (TMA box), so
// no weight byte is read twice.  GU / DN: one full 128-row weight tile per CTA and a slice of the
// contraction; the slices of a tile are added, in slice order, by the last of its CTAs to arrive.
// A kernel launched with programmatic stream serialisation starts fetching its weights while
// the previous kernel drains: only the activation fetches and the epilogue wait for it.
#include <cuda_fp16.h>
#include <string.h>

#include <atomic>

#include "tc_common.cuh"

namespace mrp {
namespace {

constexpr int kSkThreads = 192;
constexpr int kWTile = 128 * 128;          // bytes of a 128-row weight tile of one k-chunk
constexpr int kAuxBytes = 12288;           // epilogue scratch after the barriers
constexpr int kAuxRstd = 0;                // float[128]
constexpr int kAuxRowOff = 512;            // long long[32]
constexpr int kAuxVote = 768;              // int: epilogue warps' common decision
constexpr int kAuxSsq = 1024;              // float[4][128]
constexpr int kAuxExch = 4096;             // float[16][64]

enum { SK_GU = 0, SK_DN = 1, SK_LM = 2, SK_LIN = 3 };

struct SkMaps {
    CUtensorMap x;      // activation operand, box = r_pad rows
    CUtensorMap w[6];   // w[0] = 128-row tiles of gate / the matrix, w[3] = 128-row tiles of up;
                        // w[1], w[2], w[4], w[5] = LM tiles of the other heights (lm_h[0..3])
};

struct SkParams {
    int units_total;     // weight rows / 16 (GU: gate rows / 8, a unit = 8 gate + 8 up rows)
    int k_chunks;        // contraction extent / 64
    int n_stages;
    int kc;              // 64-element k-chunks per ring stage
    int r_pad;           // activation rows per part (16, 32, 64 or 128; LM: 16 or 32); MMA N = n_parts * r_pad
    int n_parts;         // operand parts stacked on N: 2 (bf16 hi + lo) or 4 (e4m3 limbs)
    int tmem_cols;       // allocated TMEM columns (power of two >= 2 buffers * 2 * r_pad)
    int lo_x, lo_xt;     // row offset of the lo block in the head operands / the LM-head operand
    int lm_h[4];         // LM: tile heights (units) other than 8, fetched through maps w[1], w[2], w[4], w[5]
    int n_split;         // GU/DN: CTAs sharing one 128-row weight tile, each a slice of the contraction
    int w_rows;          // GU/DN: weight rows (gate rows for GU)
    float *scratch;      // GU/DN: partial accumulators [tile][split][RP][128]
    int32_t *counters;   // GU/DN: arrivals per tile (zero between launches)
    int M, K, V, d, F, n_rs;
    // LM
    const float *logits0;
    const int32_t *row_index;
    int n_rows_in;       // row_index entries at or above are invalid: their base logits read as zero
    int l0_bf16;         // logits0 holds bf16 values
    Partial *partials;
    float *logits_out;
    // GU
    const float *sumsq;
    int n_ss;
    float eps;
    __nv_bfloat16 *act;
    // DN
    float *hcur;
    const float *h0f;
    const __nv_bfloat16 *gamma_next;
    __nv_bfloat16 *xg_next;
    __nv_bfloat16 *xt_k;
    __half *xt16_k;      // optional: the same rows rounded once to fp16 (fp16 LM-head mode)
    float *sumsq_out;
    float *hidden_out;
    // LIN: a plain product on operands of the caller's own (the module): out[m, j] (+)= rstd(m) * sum, rstd from
    // `sumsq` (as GU) or 1; with xg_next also out * gamma_next as the next operand and partial sums of squares of out
    float *lin_out;
    int lin_n_out;       // row pitch of lin_out and of xg_next
    int lin_accumulate;
    // LIN over lin_nw = 3 matrices of one shape sharing the operand rows (q, k, v): lin_tiles_w tiles each, through
    // maps w[0], w[1], w[2], results to lin_out, lin_out1, lin_out2
    int lin_nw, lin_tiles_w;
    float *lin_out1, *lin_out2;
    int32_t *status;
    int32_t *user_status;
    // LM with 8-bit weights: per-vocabulary-row scales of the e4m3 copy of W_lm, per-row-step scales of
    // the operand's e4m3 limbs
    const float *w8_scale;
    const float *x8_scale;
};

__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

__device__ __forceinline__ void store_hi_lo(__nv_bfloat16 *dst, size_t lo_off, float v)
{
    const __nv_bfloat16 hi = __float2bfloat16_rn(v);
    dst[0] = hi;
    dst[lo_off] = __float2bfloat16_rn(v - __bfloat162float(hi));
}

// KC: k-chunks (128 bytes of every row) per ring stage (2 for the LM head: fewer, larger stages stream better).
// FP8 (LM head only): the weights are an e4m3 copy of W_lm with one power-of-two scale per row, a k-chunk
// is 128 elements, and the activation operand is four e4m3 limbs per row-step (x = t * sum_i 16^-i limb_i,
// exact to 2^-16) stacked on N instead of the bf16 hi + lo pair.
template <int KIND, int RP, bool MARGIN, int KC, bool FP8 = false>
__global__ void __launch_bounds__(kSkThreads, 1)
sk_gemm_kernel(const __grid_constant__ SkMaps maps, const SkParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    constexpr int NP = FP8 ? 4 : 2;                  // operand parts stacked on N: 4 limbs, or hi and lo
    constexpr int kElem = FP8 ? 128 : kBK;           // elements of the contraction per k-chunk
    constexpr int x_bytes = NP * RP * 128;           // the parts' rows of one k-chunk
    constexpr int sub_bytes = kWTile + x_bytes;      // one k-chunk: weight tile, then activation rows
    constexpr int stage_bytes = KC * sub_bytes;
    const uint32_t bars = base + (uint32_t)p.n_stages * stage_bytes;
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (p.n_stages + s); };
    auto tfull_bar = [&](int a) { return bars + 8u * (2 * p.n_stages + a); };
    auto tempty_bar = [&](int a) { return bars + 8u * (2 * p.n_stages + 2 + a); };
    uint8_t *gen_base = smem_raw + (base - smem_u32(smem_raw));
    uint8_t *after_bars = gen_base + (size_t)p.n_stages * stage_bytes + 8 * (2 * p.n_stages + 4);
    uint32_t *tmem_holder = reinterpret_cast<uint32_t *>(after_bars);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_holder + 1);
    uint8_t *aux = after_bars + 16;        // 16-byte aligned: stages and barrier block are multiples of 16

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int cta = blockIdx.x, G = gridDim.x;
    // LM: a contiguous range of 16-row units per CTA, the whole contraction.
    // GU/DN: one full 128-row tile per CTA and one of n_split slices of the contraction; the
    // slices of a tile are summed, in slice order, by whichever of its CTAs finishes last.
    int units, u0, kc0 = 0, kc1 = p.k_chunks;
    if (KIND == SK_LM) {
        const int u_base = p.units_total / G, u_extra = p.units_total % G;
        units = u_base + (cta < u_extra ? 1 : 0);
        u0 = cta * u_base + min(cta, u_extra);
    } else {
        const int cps = (p.k_chunks + p.n_split - 1) / p.n_split;
        units = 8;
        u0 = (cta / p.n_split) * 8;
        if (KIND == SK_LIN && p.lin_nw == 3) u0 = ((cta / p.n_split) % p.lin_tiles_w) * 8;
        kc0 = (cta % p.n_split) * cps;
        kc1 = min(p.k_chunks, kc0 + cps);
    }
    const int nk = (kc1 - kc0) / KC;                 // ring stages per tile
    // The range is cut into the fewest tiles of at most 8 units and the tiles are made equally
    // high (an MMA costs the same at any height, so a short extra tile would cost a full one):
    // the first t_extra tiles have t_base + 1 units, the others t_base.
    const int n_tiles = (units + 7) >> 3;
    const int t_base = n_tiles ? units / n_tiles : 0, t_extra = n_tiles ? units % n_tiles : 0;
    auto tile_units = [&](int ti) { return t_base + (ti < t_extra ? 1 : 0); };
    auto tile_start = [&](int ti) { return u0 + ti * t_base + min(ti, t_extra); };
    auto tile_map = [&](int h) {
        if (h == 8) return 0;
        return h == p.lm_h[0] ? 1 : h == p.lm_h[1] ? 2 : h == p.lm_h[2] ? 4 : 5;
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.n_stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 4); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        prefetch_tmap(&maps.x);
        prefetch_tmap(&maps.w[0]);
        if (KIND == SK_GU) prefetch_tmap(&maps.w[3]);
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_holder)), "r"((uint32_t)p.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;
    griddep_launch();

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            const int total_it = n_tiles * nk;
            const int pre = min(p.n_stages, total_it);
            const uint64_t pol_w = l2_policy_evict_first(), pol_x = l2_policy_evict_last();
            auto load_w = [&](int t, int kk, int s) {
                const uint32_t sw = base + (uint32_t)s * stage_bytes;
                const int h = tile_units(t);
                mbar_expect_tx(full_bar(s), (uint32_t)KC * ((uint32_t)h * 2048u + (uint32_t)x_bytes));
                const int ut = tile_start(t);
#pragma unroll
                for (int b = 0; b < KC; ++b) {
                    const int kx = (kc0 + kk * KC + b) * kElem;
                    if (KIND == SK_GU) {
                        tma_load_2d_hint(sw + b * sub_bytes, &maps.w[0], kx, ut * 8, full_bar(s), pol_w);
                        tma_load_2d_hint(sw + b * sub_bytes + 64 * 128, &maps.w[3], kx, ut * 8, full_bar(s), pol_w);
                    } else {
                        const int mi = (KIND == SK_LIN && p.lin_nw == 3) ? (cta / p.n_split) / p.lin_tiles_w : tile_map(h);
                        tma_load_2d_hint(sw + b * sub_bytes, &maps.w[mi], kx, ut * 16, full_bar(s), pol_w);
                    }
                }
            };
            auto load_x = [&](int kk, int s) {
                const uint32_t sx = base + (uint32_t)s * stage_bytes + kWTile;
                // one box per k-chunk: RP hi rows, then (the lo block starts at row RP of the buffer) RP lo rows
#pragma unroll
                for (int b = 0; b < KC; ++b)
                    tma_load_2d_hint(sx + b * sub_bytes, &maps.x, (kc0 + kk * KC + b) * kElem, 0, full_bar(s), pol_x);
            };
            // weights do not depend on the previous kernel: fill the ring with them first
            int t = 0, kk = 0;
            for (int it = 0; it < pre; ++it) {
                load_w(t, kk, it);
                if (++kk == nk) { kk = 0; ++t; }
            }
            griddep_wait();
            for (int it = 0, k2 = 0; it < pre; ++it) {
                load_x(k2, it);
                if (++k2 == nk) k2 = 0;
            }
            int s = 0;
            uint32_t ph = 1;              // the ring has been filled once
            for (int it = pre; it < total_it; ++it) {
                if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, p)) break;
                load_w(t, kk, s);
                load_x(kk, s);
                if (++kk == nk) { kk = 0; ++t; }
                if (++s == p.n_stages) { s = 0; ph ^= 1u; }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        // The whole warp walks the loop (all values are warp-uniform); the elected lane issues.
        const uint32_t idesc = FP8 ? make_idesc_e4m3(NP * RP) : make_idesc(NP * RP);
        const uint32_t tm = __shfl_sync(0xffffffffu, tmem_base, 0);
        int s = 0, acc = 0;
        uint32_t ph = 0, acc_ph = 0;
        bool ok = true;
        for (int t = 0; t < n_tiles && ok; ++t) {
            ok = __all_sync(0xffffffffu, mbar_wait(tempty_bar(acc), acc_ph ^ 1u, abort_flag, p));
            if (!ok) break;
            tc_fence_after();
            const uint32_t dt = tm + (uint32_t)(acc * NP * RP);
            for (int kk = 0; kk < nk; ++kk) {
                const uint32_t sw = base + (uint32_t)s * stage_bytes;
                const uint32_t later = kk > 0 ? 1u : 0u;
                ok = __all_sync(0xffffffffu, mbar_wait(full_bar(s), ph, abort_flag, p));
                if (!ok) break;
                tc_fence_after();
                if (elect_one()) {
#pragma unroll
                    for (int b = 0; b < KC; ++b) {
                        const uint64_t dw = make_smem_desc(sw + b * sub_bytes);
                        const uint64_t dx = make_smem_desc(sw + b * sub_bytes + kWTile);
#pragma unroll
                        for (int k4 = 0; k4 < 4; ++k4) {         // 32 bytes of every row per MMA
                            if (FP8) umma_f8(dt, dw + 2u * k4, dx + 2u * k4, idesc, (b > 0 || k4 > 0) ? 1u : later);
                            else umma_bf16(dt, dw + 2u * k4, dx + 2u * k4, idesc, (b > 0 || k4 > 0) ? 1u : later);
                        }
                    }
                    umma_commit(empty_bar(s));
                }
                __syncwarp();
                if (++s == p.n_stages) { s = 0; ph ^= 1u; }
            }
            if (!ok) break;
            if (elect_one()) umma_commit(tfull_bar(acc));
            __syncwarp();
            acc ^= 1;
            if (acc == 0) acc_ph ^= 1u;
        }
    } else {
        // ---------------- epilogue warps: thread t owns TMEM lane t = weight row t of the tile ----
        const int q = warp & 3;
        const int t = q * 32 + lane;
        const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
        float *rstd_s = reinterpret_cast<float *>(aux + kAuxRstd);
        long long *rowoff_s = reinterpret_cast<long long *>(aux + kAuxRowOff);
        float *ssq_s = reinterpret_cast<float *>(aux + kAuxSsq);
        float *exch_s = reinterpret_cast<float *>(aux + kAuxExch);
        volatile int *vote_s = reinterpret_cast<volatile int *>(aux + kAuxVote);

        if (t == 0) *vote_s = 0;
        griddep_wait();
        if (KIND == SK_LM) {
            if (FP8 && t < RP) rstd_s[t] = t < p.n_rs ? p.x8_scale[t] : 0.f;     // the limbs' per-row-step scales
            if (t < p.n_rs) {
                const int m = t % p.M;
                const int idx = p.row_index ? p.row_index[m] : m;
                // -1: no base logits for this row-step (none given, or the caller's index is out of range)
                rowoff_s[t] = (p.logits0 && (!p.row_index || row_ok(idx, p.n_rows_in))) ? (long long)idx * p.V : -1ll;
            }
        } else if (KIND == SK_GU || KIND == SK_LIN) {
            if (t < p.M) {
                float s = 0.f;
                if (KIND == SK_GU || p.sumsq)
                    for (int i = 0; i < p.n_ss; ++i) s += p.sumsq[(size_t)i * p.M + t];
                rstd_s[t] = (KIND == SK_GU || p.sumsq) ? rsqrtf(s / (float)p.d + p.eps) : 1.f;
            }
        }
        epi_sync();

        if constexpr (KIND == SK_LM) {
            // per-thread running statistics of every row-step
            float st_mx[RP], st_sum[RP], st_sec[RP];
            int st_idx[RP];
#pragma unroll
            for (int s = 0; s < RP; ++s) { st_mx[s] = -INFINITY; st_sum[s] = 0.f; st_sec[s] = -INFINITY; st_idx[s] = INT_MAX; }
            int acc = 0;
            uint32_t acc_ph = 0;
            bool ok = true;
            for (int ti = 0; ti < n_tiles && ok; ++ti) {
                const int ut = tile_start(ti);
                const int units_here = tile_units(ti);
                const int v = ut * 16 + t;
                const bool valid = t < units_here * 16;
                // What the tile's outputs are added to does not depend on the accumulator: fetch
                // it (independent loads, all in flight together) before waiting for the MMAs.
                float a[RP];
#pragma unroll
                for (int j = 0; j < RP; ++j)
                    a[j] = (valid && j < p.n_rs && rowoff_s[j] >= 0) ? ld_l0(p.logits0, p.l0_bf16, (size_t)(rowoff_s[j] + v)) : 0.f;
                float ws = 0.f;                              // 8-bit weights: the scale of this thread's vocabulary row
                if (FP8 && valid) ws = __ldg(p.w8_scale + v);
                ok = __all_sync(0xffffffffu, mbar_wait(tfull_bar(acc), acc_ph, abort_flag, p));
                if (!ok) break;
                tc_fence_after();
                const uint32_t tacc = lane_addr + (uint32_t)(acc * NP * RP);
                if constexpr (!FP8) {
#pragma unroll
                    for (int c0 = 0; c0 < 2 * RP; c0 += 16) {          // products with the hi rows, then the lo rows
                        float part[16];
                        tmem_ld16(tacc + c0, part);
#pragma unroll
                        for (int j = 0; j < 16; ++j) a[(c0 + j) % RP] += part[j];
                    }
                } else {
                    // delta = (row scale of W) * (scale of the row-step) * sum_i 16^-i (W8 . limb_i)
                    float dsum[RP];
#pragma unroll
                    for (int j = 0; j < RP; ++j) dsum[j] = 0.f;
#pragma unroll
                    for (int c0 = 0; c0 < 4 * RP; c0 += 16) {
                        float part[16];
                        tmem_ld16(tacc + c0, part);
                        const float lw = (c0 / RP) == 0 ? 1.f : (c0 / RP) == 1 ? 0.0625f : (c0 / RP) == 2 ? 0.00390625f : 0.000244140625f;
#pragma unroll
                        for (int j = 0; j < 16; ++j) dsum[(c0 + j) % RP] = fmaf(part[j], lw, dsum[(c0 + j) % RP]);
                    }
#pragma unroll
                    for (int j = 0; j < RP; ++j) a[j] = fmaf(dsum[j], ws * rstd_s[j], a[j]);
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(tempty_bar(acc));
                acc ^= 1;
                if (acc == 0) acc_ph ^= 1u;
                if (valid) {
#pragma unroll
                    for (int s = 0; s < RP; ++s) {
                        if (s < p.n_rs) {
                            const float l = a[s];
                            const float nm = fmaxf(st_mx[s], l);
                            st_sum[s] = st_sum[s] * ex2f((st_mx[s] - nm) * kLog2e) + ex2f((l - nm) * kLog2e);
                            if (l > st_mx[s]) {
                                if (MARGIN) st_sec[s] = st_mx[s];
                                st_idx[s] = v;
                            } else if (MARGIN) {
                                st_sec[s] = fmaxf(st_sec[s], l);
                            }
                            st_mx[s] = nm;
                            if (p.logits_out && s >= p.M) p.logits_out[(size_t)(s - p.M) * p.V + v] = l;
                        }
                    }
                }
            }
            // Every thread parks its row-step statistics in the (now idle) ring memory; the merge
            // over the 128 threads is then a short loop instead of unrolled straight-line code,
            // which would be fetched once, instruction line by line, from a saturated memory system.
            Partial *park = reinterpret_cast<Partial *>(gen_base);
            if (!ok && lane == 0) *vote_s = 1;
            epi_sync();
            ok = (*vote_s == 0);          // on a failed wait copies may still be landing in the ring
            if (ok) {
#pragma unroll
                for (int s = 0; s < RP; ++s) {
                    if (s < p.n_rs) {
                        Partial pr;
                        pr.mx = st_mx[s]; pr.sum = st_sum[s]; pr.idx = st_idx[s]; pr.second = st_sec[s];
                        park[s * 128 + t] = pr;
                    }
                }
            }
            epi_sync();
            if (ok) {
#pragma unroll 1
                for (int s = q; s < p.n_rs; s += 4) {
                    // fixed order: lane quadrants first, then the butterfly over lanes
                    Partial pr = park[s * 128 + lane];
#pragma unroll 1
                    for (int w = 1; w < 4; ++w) pr = merge_partial(pr, park[s * 128 + w * 32 + lane]);
#pragma unroll 1
                    for (int o = 16; o > 0; o >>= 1) {
                        Partial other;
                        other.mx = __shfl_xor_sync(0xffffffffu, pr.mx, o);
                        other.sum = __shfl_xor_sync(0xffffffffu, pr.sum, o);
                        other.idx = __shfl_xor_sync(0xffffffffu, pr.idx, o);
                        other.second = __shfl_xor_sync(0xffffffffu, pr.second, o);
                        pr = (lane & o) ? merge_partial(other, pr) : merge_partial(pr, other);
                    }
                    if (lane == 0) p.partials[(size_t)cta * p.n_rs + s] = pr;
                }
            }
        } else {
            // GU / DN: one weight tile per CTA; activation columns are handled 16 at a time
            const int wrow = KIND == SK_GU ? u0 * 8 + t : u0 * 16 + t;     // weight row = output feature
            const bool valid = KIND == SK_GU ? (t < 64 && wrow < p.w_rows) : (wrow < p.w_rows);
            const int n_ch = (p.M + 15) >> 4;
            const int tile = cta / p.n_split;
            const int which = (KIND == SK_LIN && p.lin_nw == 3) ? tile / p.lin_tiles_w : 0;
            float *lin_dst = which == 0 ? p.lin_out : which == 1 ? p.lin_out1 : p.lin_out2;
            bool ok = __all_sync(0xffffffffu, mbar_wait(tfull_bar(0), 0u, abort_flag, p));
            // the four warps meet at barriers below: they must agree on going on
            if (!ok && lane == 0) *vote_s = 1;
            epi_sync();
            ok = (*vote_s == 0);
            bool finisher = ok;
            if (ok) tc_fence_after();
            if (ok && p.n_split > 1) {
                // park this slice's partial sums; the last CTA of the tile to arrive adds the slices
                float *mine = p.scratch + ((size_t)cta * RP) * 128;
#pragma unroll 1
                for (int ch = 0; ch < n_ch; ++ch) {
                    float v[16], w[16];
                    tmem_ld16(lane_addr + ch * 16, v);
                    tmem_ld16(lane_addr + RP + ch * 16, w);
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        if (ch * 16 + j < p.M) mine[(ch * 16 + j) * 128 + t] = v[j] + w[j];
                }
                // one thread's fence after the barrier publishes every thread's stores (fences are cumulative)
                epi_sync();
                if (t == 0) {
                    __threadfence();
                    *vote_s = (atomicAdd(p.counters + tile, 1) == p.n_split - 1) ? 2 : 0;
                }
                epi_sync();
                finisher = (*vote_s == 2);
                if (finisher) {
                    __threadfence();
                    if (t == 0) p.counters[tile] = 0;
                }
            }
            if (finisher) {
                const float *first = p.scratch + ((size_t)tile * p.n_split * RP) * 128;
                const float gm = ((KIND == SK_DN || KIND == SK_LIN) && valid && p.xg_next) ? __bfloat162float(p.gamma_next[wrow]) : 0.f;
#pragma unroll 1
                for (int ch = 0; ch < n_ch; ++ch) {
                    const int c0 = ch * 16;
                    float v[16];
                    float hc[16], h0v[16];          // DN: what the outputs are added to, fetched first
                    if (KIND == SK_DN) {
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            hc[j] = 0.f; h0v[j] = 0.f;
                            if (valid && c0 + j < p.M) {
                                hc[j] = p.hcur[(size_t)(c0 + j) * p.d + wrow];
                                h0v[j] = __ldg(p.h0f + (size_t)(c0 + j) * p.d + wrow);
                            }
                        }
                    }
                    if (p.n_split > 1) {
#pragma unroll
                        for (int j = 0; j < 16; ++j) v[j] = 0.f;
#pragma unroll 4
                        for (int sp = 0; sp < p.n_split; ++sp) {   // slice order: the sum does not depend on who is last
#pragma unroll
                            for (int j = 0; j < 16; ++j)
                                if (c0 + j < p.M) v[j] += __ldcg(first + ((size_t)sp * RP + c0 + j) * 128 + t);
                        }
                    } else {
                        float w[16];
                        tmem_ld16(lane_addr + c0, v);
                        tmem_ld16(lane_addr + RP + c0, w);
#pragma unroll
                        for (int j = 0; j < 16; ++j) v[j] += w[j];
                    }
                    if (KIND == SK_GU) {
                        // lanes 0-63 hold gate rows, 64-127 the matching up rows: hand the up values over
                        if (t >= 64) {
#pragma unroll
                            for (int j = 0; j < 16; ++j)
                                if (c0 + j < p.M) exch_s[j * 64 + (t - 64)] = v[j] * rstd_s[c0 + j];
                        }
                        epi_sync();
                        if (valid) {
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                if (c0 + j < p.M) {
                                    const float g = v[j] * rstd_s[c0 + j];
                                    const float av = g / (1.f + __expf(-g)) * exch_s[j * 64 + t];
                                    store_hi_lo(p.act + (size_t)(c0 + j) * p.F + wrow, (size_t)p.lo_x * p.F, av);
                                }
                            }
                        }
                        epi_sync();
                    } else if (KIND == SK_LIN) {
                        float sq[16];
#pragma unroll
                        for (int j = 0; j < 16; ++j) sq[j] = 0.f;
                        if (valid) {
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                if (c0 + j < p.M) {
                                    const size_t o = (size_t)(c0 + j) * p.lin_n_out + wrow;
                                    float h = v[j] * rstd_s[c0 + j];
                                    if (p.lin_accumulate) h += lin_dst[o];
                                    lin_dst[o] = h;
                                    sq[j] = h * h;
                                    if (p.xg_next) store_hi_lo(p.xg_next + o, (size_t)p.lo_x * p.lin_n_out, h * gm);
                                }
                            }
                        }
                        if (p.xg_next) {
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                float s = sq[j];
#pragma unroll
                                for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
                                if (lane == 0) ssq_s[q * 128 + c0 + j] = s;
                            }
                        }
                    } else {
                        float sq[16];
#pragma unroll
                        for (int j = 0; j < 16; ++j) sq[j] = 0.f;
                        if (valid) {
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                if (c0 + j < p.M) {
                                    const size_t o = (size_t)(c0 + j) * p.d + wrow;
                                    const float h = hc[j] + v[j];
                                    p.hcur[o] = h;
                                    if (p.hidden_out) p.hidden_out[o] = h;
                                    sq[j] = h * h;
                                    store_hi_lo(p.xt_k + o, (size_t)p.lo_xt * p.d, h - h0v[j]);
                                    if (p.xt16_k) p.xt16_k[o] = __float2half_rn(h - h0v[j]);
                                    if (p.xg_next) store_hi_lo(p.xg_next + o, (size_t)p.lo_x * p.d, h * gm);
                                }
                            }
                        }
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            float s = sq[j];
#pragma unroll
                            for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
                            if (lane == 0) ssq_s[q * 128 + c0 + j] = s;
                        }
                    }
                }
            }
            if (KIND == SK_DN || (KIND == SK_LIN && p.xg_next)) {
                epi_sync();
                // one slice of sums of squares per weight tile, written by the CTA that finished it
                if (finisher) {
                    for (int m = t; m < p.M; m += 128)
                        p.sumsq_out[(size_t)tile * p.M + m] =
                            (ssq_s[m] + ssq_s[128 + m]) + (ssq_s[256 + m] + ssq_s[384 + m]);
                }
            }
        }
    }

    // ---------------- teardown ----------------
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        // a wait gave up: give copies still in flight time to land before the CTA leaves
        const long long t0 = clock64();
        while (clock64() - t0 < 200000) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)p.tmem_cols) : "memory");
    }
}

// ---------------------------------------------------------------------------------------
// 8-bit LM head: quantiser of W_lm (once, at context creation) and of the operand rows (every call)
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ float block_max(float v, float *red)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float m = 0.f;
    for (int i = 0; i < (int)(blockDim.x >> 5); ++i) m = fmaxf(m, red[i]);
    __syncthreads();
    return m;
}

// One block per vocabulary row: scale = 2^E with max|row| <= 448 * 2^E, codes = e4m3(row / scale).
__global__ void quantise_rows_kernel(const __nv_bfloat16 *__restrict__ w, int d, uint8_t *__restrict__ codes,
                                     float *__restrict__ scales)
{
    __shared__ float red[32];
    const size_t row = blockIdx.x;
    float amax = 0.f;
    for (int j = threadIdx.x; j < d; j += blockDim.x) amax = fmaxf(amax, fabsf(__bfloat162float(w[row * d + j])));
    amax = block_max(amax, red);
    const float sc = e4m3_row_scale(amax), inv = 1.f / sc;       // a power of two: the division is exact
    if (threadIdx.x == 0) scales[row] = sc;
    for (int j = threadIdx.x; j < d; j += blockDim.x)
        codes[row * d + j] = (uint8_t)f32_to_e4m3(__bfloat162float(w[row * d + j]) * inv);
}

// One block per row-step of the stacked LM-head operand (bf16 hi + lo rows): x = t * (l_0 + l_1 / 16 +
// l_2 / 256 + l_3 / 4096), t a power of two, every l_i an e4m3 value: each limb takes what the
// previous ones left (the subtractions are exact in fp32), so x is met to 2^-16 relative.
// Limb i of row-step r is row i * r_pad + r of xq.
__global__ void operand_limbs_kernel(const __nv_bfloat16 *__restrict__ xt, int lo_rows, int d, int r_pad,
                                     uint8_t *__restrict__ xq, float *__restrict__ x_scale)
{
    pdl_trigger();
    pdl_wait();
    __shared__ float red[32];
    const int r = blockIdx.x;
    const __nv_bfloat16 *hi = xt + (size_t)r * d, *lo = xt + ((size_t)lo_rows + r) * d;
    float amax = 0.f;
    for (int j = threadIdx.x; j < d; j += blockDim.x)
        amax = fmaxf(amax, fabsf(__bfloat162float(hi[j]) + __bfloat162float(lo[j])));
    amax = block_max(amax, red);
    const float sc = e4m3_row_scale(amax), inv = 1.f / sc;
    if (threadIdx.x == 0) x_scale[r] = sc;
    for (int j = threadIdx.x; j < d; j += blockDim.x) {
        float y = (__bfloat162float(hi[j]) + __bfloat162float(lo[j])) * inv;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t q = f32_to_e4m3(y);
            xq[((size_t)i * r_pad + r) * d + j] = (uint8_t)q;
            y = (y - e4m3_to_f32(q)) * 16.f;
        }
    }
}

// ---------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------
size_t sk_smem_bytes(const SkParams &p)
{
    const int stage = p.kc * (kWTile + p.n_parts * p.r_pad * 128);
    return (size_t)p.n_stages * stage + 1024 + 8 * (2 * p.n_stages + 4) + 16 + kAuxBytes;
}

void sk_finish_shape(SkParams &p, int grid)
{
    // the ring always takes all the shared memory there is: it also parks the LM statistics
    if (p.kc < 1) p.kc = 1;
    if (p.n_parts < 2) p.n_parts = 2;
    const int stage = p.kc * (kWTile + p.n_parts * p.r_pad * 128);
    int ns = (kSmemBudget - 1024 - 256 - 16 - kAuxBytes) / stage;
    if (ns > 12) ns = 12;
    p.n_stages = ns;
    int cols = 32;
    while (cols < 2 * p.n_parts * p.r_pad) cols <<= 1;
    p.tmem_cols = cols;
    p.n_split = 1;
    for (int i = 0; i < 4; ++i) p.lm_h[i] = 0;
    if (grid > 0) {           // LM: contiguous unit ranges of u_base or u_base + 1 units, equal-height tiles
        int n = 0;
        for (int units = p.units_total / grid; units <= p.units_total / grid + 1; ++units) {
            const int nt = (units + 7) / 8;
            if (nt == 0) continue;
            for (int h = units / nt; h <= units / nt + (units % nt ? 1 : 0); ++h) {
                bool seen = (h == 8 || h == 0);
                for (int i = 0; i < n; ++i) seen |= (p.lm_h[i] == h);
                if (!seen) p.lm_h[n++] = h;
            }
        }
    }
}

// GU/DN: n_tiles full weight tiles, each shared by n_split CTAs that take slices of the contraction.
int sk_split(Ctx *c, SkParams &p, int n_tiles)
{
    int S = c->sm_count / n_tiles;
    if (S < 1) S = 1;
    if (S > p.k_chunks) S = p.k_chunks;
    const int cps = (p.k_chunks + S - 1) / S;
    S = (p.k_chunks + cps - 1) / cps;          // no empty slice
    if ((size_t)n_tiles * S * p.r_pad * 128 * 4 > (size_t)kSkScratchBytes) S = 1;
    p.n_split = S;
    p.scratch = (float *)(c->ws + c->lay.sk_scratch);
    p.counters = (int32_t *)(c->ws + c->lay.sk_counters);
    return n_tiles * S;
}

// Tensor maps of one weight matrix part: full tiles, and for the LM head the other tile heights.
bool sk_weight_maps(const TcState *s, SkMaps &maps, int part, const void *w, uint64_t inner, uint64_t rows,
                    int unit_rows, const SkParams &p)
{
    if (!make_map(s, &maps.w[part * 3], w, inner, rows, 8 * unit_rows)) return false;
    static const int slot[4] = {1, 2, 4, 5};
    for (int k = 0; k < 4 && part == 0; ++k)
        if (p.lm_h[k] > 0 && !make_map(s, &maps.w[slot[k]], w, inner, rows, p.lm_h[k] * unit_rows)) return false;
    return true;
}

template <int KIND, int RP, bool MARGIN, int KC = 1, bool FP8 = false>
cudaError_t sk_launch(const SkMaps &maps, const SkParams &p, int grid, cudaStream_t st, bool pdl)
{
    auto kern = sk_gemm_kernel<KIND, RP, MARGIN, KC, FP8>;
    // the shared-memory limit of a kernel is set once per device (the attribute is per device)
    static std::atomic<unsigned long long> attr_devices{0};
    int dev = 0;
    cudaError_t ea = cudaGetDevice(&dev);
    if (ea != cudaSuccess) return ea;
    const unsigned long long bit = 1ull << (dev & 63);
    if (!(attr_devices.load() & bit)) {
        ea = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
        if (ea != cudaSuccess) return ea;
        attr_devices.fetch_or(bit);
    }
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kSkThreads);
    cfg.dynamicSmemBytes = sk_smem_bytes(p);
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, maps, p);
}

template <int KIND>
cudaError_t sk_launch_rp(const SkMaps &maps, const SkParams &p, int grid, cudaStream_t st, bool pdl, bool margin)
{
    if constexpr (KIND != SK_LM) {
        switch (p.r_pad) {
        case 16: return sk_launch<KIND, 16, false>(maps, p, grid, st, pdl);
        case 32: return sk_launch<KIND, 32, false>(maps, p, grid, st, pdl);
        case 64: return sk_launch<KIND, 64, false>(maps, p, grid, st, pdl);
        default: return sk_launch<KIND, 128, false>(maps, p, grid, st, pdl);
        }
    } else {
        if (p.n_parts == 4) {       // e4m3 weights and operand limbs (two k-chunks per stage)
            if (p.r_pad == 16)
                return margin ? sk_launch<KIND, 16, true, 2, true>(maps, p, grid, st, pdl) : sk_launch<KIND, 16, false, 2, true>(maps, p, grid, st, pdl);
            return margin ? sk_launch<KIND, 32, true, 2, true>(maps, p, grid, st, pdl) : sk_launch<KIND, 32, false, 2, true>(maps, p, grid, st, pdl);
        }
        if (p.kc == 2) {
            if (p.r_pad == 16)
                return margin ? sk_launch<KIND, 16, true, 2>(maps, p, grid, st, pdl) : sk_launch<KIND, 16, false, 2>(maps, p, grid, st, pdl);
            return margin ? sk_launch<KIND, 32, true, 2>(maps, p, grid, st, pdl) : sk_launch<KIND, 32, false, 2>(maps, p, grid, st, pdl);
        }
        if (p.r_pad == 16)
            return margin ? sk_launch<KIND, 16, true>(maps, p, grid, st, pdl) : sk_launch<KIND, 16, false>(maps, p, grid, st, pdl);
        return margin ? sk_launch<KIND, 32, true>(maps, p, grid, st, pdl) : sk_launch<KIND, 32, false>(maps, p, grid, st, pdl);
    }
}

void sk_common(Ctx *c, SkParams &p, int M, int K, const mrp_draft_out &out)
{
    memset(&p, 0, sizeof(p));
    p.M = M; p.K = K; p.V = c->cfg.vocab; p.d = c->cfg.d; p.F = c->cfg.d_ff; p.n_rs = (K + 1) * M;
    p.status = (int32_t *)(c->ws + c->lay.status);
    p.user_status = out.status;
    p.lo_x = c->lo_x; p.lo_xt = c->lo_xt;
}

}  // namespace

int sk_head_pad(int M) { return M <= 16 ? 16 : M <= 32 ? 32 : M <= 64 ? 64 : 128; }

int sk_lm_pad(int n_rs) { return n_rs <= 16 ? 16 : 32; }

bool sk_rows_ok(int rows) { return rows >= 1 && rows <= 32; }

// Above 64 rows the per-CTA re-read of the activation tile and the serial 16-column epilogue
// cost more than the row-major kernels' narrow weight tiles (measured at M = 128).
bool sk_head_rows_ok(int M) { return M >= 1 && M <= 64; }

bool sk_heads_ok(const mrp_config &cfg) { return (cfg.d + 127) / 128 <= kSumsqSlices && cfg.d_ff / 64 < kSkMaxTiles; }

cudaError_t sk_gateup(Ctx *c, int k, int M, int K, int n_ss, const mrp_draft_out &out, cudaStream_t st, bool pdl)
{
    const TcState *s = (const TcState *)c->tc_state;
    const mrp_head_weights &hw = c->heads[k - 1];
    const int d = c->cfg.d, F = c->cfg.d_ff, G = c->sm_count;
    SkParams p;
    sk_common(c, p, M, K, out);
    p.units_total = F / 8; p.k_chunks = d / kBK; p.r_pad = sk_head_pad(M); p.w_rows = F;
    p.sumsq = (const float *)(c->ws + c->lay.sumsq); p.n_ss = n_ss; p.eps = c->cfg.rms_eps;
    p.act = (__nv_bfloat16 *)(c->ws + c->lay.act);
    sk_finish_shape(p, 0);
    const int grid = sk_split(c, p, F / 64);
    (void)G;
    SkMaps maps;
    memset(&maps, 0, sizeof(maps));
    if (!make_map(s, &maps.x, c->ws + c->lay.xg, d, 2 * (uint64_t)p.r_pad, 2 * p.r_pad) ||
        !sk_weight_maps(s, maps, 0, hw.w_gate, d, F, 8, p) || !sk_weight_maps(s, maps, 1, hw.w_up, d, F, 8, p))
        return note_err(c, cudaErrorInvalidValue, "tensor map (gate/up, few rows)");
    c->launches++;
    return note_err(c, sk_launch_rp<SK_GU>(maps, p, grid, st, pdl, false), "gate/up kernel (few rows)");
}

cudaError_t sk_down(Ctx *c, int k, int M, int K, const mrp_draft_out &out, cudaStream_t st, bool pdl, int *n_ss_out,
                    bool f16_lm)
{
    const TcState *s = (const TcState *)c->tc_state;
    const mrp_head_weights &hw = c->heads[k - 1];
    const int d = c->cfg.d, F = c->cfg.d_ff, G = c->sm_count;
    SkParams p;
    sk_common(c, p, M, K, out);
    p.units_total = d / 16; p.k_chunks = F / kBK; p.r_pad = sk_head_pad(M); p.w_rows = d;
    p.hcur = (float *)(c->ws + c->lay.hcur); p.h0f = (const float *)(c->ws + c->lay.h0f);
    p.gamma_next = (k < K) ? (const __nv_bfloat16 *)c->heads[k].rms_gamma : nullptr;
    p.xg_next = (k < K) ? (__nv_bfloat16 *)(c->ws + c->lay.xg) : nullptr;
    p.xt_k = (__nv_bfloat16 *)(c->ws + c->lay.xt) + (size_t)k * M * d;
    p.xt16_k = f16_lm ? (__half *)(c->ws + c->lay.xt16) + (size_t)(k - (c->from_hidden ? 0 : 1)) * M * d : nullptr;
    p.sumsq_out = (float *)(c->ws + c->lay.sumsq);
    p.hidden_out = (k == K) ? out.hidden_out : nullptr;
    sk_finish_shape(p, 0);
    const int n_tiles = (d + 127) / 128;
    const int grid = sk_split(c, p, n_tiles);
    *n_ss_out = n_tiles;
    (void)G;
    SkMaps maps;
    memset(&maps, 0, sizeof(maps));
    if (!make_map(s, &maps.x, c->ws + c->lay.act, F, 2 * (uint64_t)p.r_pad, 2 * p.r_pad) ||
        !sk_weight_maps(s, maps, 0, hw.w_down, F, d, 16, p))
        return note_err(c, cudaErrorInvalidValue, "tensor map (down, few rows)");
    c->launches++;
    return note_err(c, sk_launch_rp<SK_DN>(maps, p, grid, st, pdl, false), "down kernel (few rows)");
}

// Few-row products on operands of the caller's own (the module; n <= 64 rows).  Operand a: bf16 hi rows [n, n_in]
// with the lo rows sk_head_pad(n) rows further on.
// out[n, n_out] (+)= rstd(row) * (A W^T), rstd from sumsq[n_ss, n] (nullptr: 1); with xg_next also out * gamma_next
// in operand form and partial sums of squares of out to sumsq_out[*n_ss_out, n].
cudaError_t sk_linear(Ctx *c, const __nv_bfloat16 *a, int n, int n_in, const void *w, int n_out, const float *sumsq,
                      int n_ss, float *out, bool accumulate, const void *gamma_next, __nv_bfloat16 *xg_next,
                      float *sumsq_out, int *n_ss_out, int32_t *user_status, cudaStream_t st)
{
    const TcState *s = (const TcState *)c->tc_state;
    SkParams p;
    memset(&p, 0, sizeof(p));
    p.M = n; p.d = n_in; p.F = n_in;
    p.status = (int32_t *)(c->ws + c->lay.status); p.user_status = user_status;
    p.units_total = n_out / 16; p.k_chunks = n_in / kBK; p.r_pad = sk_head_pad(n); p.w_rows = n_out;
    p.lo_x = p.r_pad; p.lo_xt = p.r_pad;
    p.sumsq = sumsq; p.n_ss = n_ss; p.eps = c->cfg.rms_eps;
    p.lin_out = out; p.lin_n_out = n_out; p.lin_accumulate = accumulate ? 1 : 0;
    p.gamma_next = (const __nv_bfloat16 *)gamma_next; p.xg_next = xg_next; p.sumsq_out = sumsq_out;
    sk_finish_shape(p, 0);
    const int n_tiles = (n_out + 127) / 128;
    const int grid = sk_split(c, p, n_tiles);
    if (n_ss_out) *n_ss_out = n_tiles;
    SkMaps maps;
    memset(&maps, 0, sizeof(maps));
    if (!make_map(s, &maps.x, a, n_in, 2 * (uint64_t)p.r_pad, 2 * p.r_pad) || !sk_weight_maps(s, maps, 0, w, n_in, n_out, 16, p))
        return note_err(c, cudaErrorInvalidValue, "tensor map (module product, few rows)");
    c->launches++;
    return note_err(c, sk_launch_rp<SK_LIN>(maps, p, grid, st, !(c->cfg.flags & MRP_FLAG_NO_PDL), false),
                    "module product kernel (few rows)");
}

// Three such products over the same operand rows in one launch (q, k, v): out_i = rstd(row) * (A W_i^T).
cudaError_t sk_linear3(Ctx *c, const __nv_bfloat16 *a, int n, int n_in, const void *w0, const void *w1, const void *w2,
                       int n_out, const float *sumsq, int n_ss, float *out0, float *out1, float *out2, int32_t *user_status,
                       cudaStream_t st)
{
    const TcState *s = (const TcState *)c->tc_state;
    SkParams p;
    memset(&p, 0, sizeof(p));
    p.M = n; p.d = n_in; p.F = n_in;
    p.status = (int32_t *)(c->ws + c->lay.status); p.user_status = user_status;
    p.units_total = n_out / 16; p.k_chunks = n_in / kBK; p.r_pad = sk_head_pad(n); p.w_rows = n_out;
    p.lo_x = p.r_pad; p.lo_xt = p.r_pad;
    p.sumsq = sumsq; p.n_ss = n_ss; p.eps = c->cfg.rms_eps;
    p.lin_out = out0; p.lin_out1 = out1; p.lin_out2 = out2; p.lin_n_out = n_out;
    sk_finish_shape(p, 0);
    const int n_tiles = (n_out + 127) / 128;
    p.lin_nw = 3; p.lin_tiles_w = n_tiles;
    const int grid = sk_split(c, p, 3 * n_tiles);
    SkMaps maps;
    memset(&maps, 0, sizeof(maps));
    if (!make_map(s, &maps.x, a, n_in, 2 * (uint64_t)p.r_pad, 2 * p.r_pad) || !make_map(s, &maps.w[0], w0, n_in, n_out, 128) ||
        !make_map(s, &maps.w[1], w1, n_in, n_out, 128) || !make_map(s, &maps.w[2], w2, n_in, n_out, 128))
        return note_err(c, cudaErrorInvalidValue, "tensor map (module q, k, v, few rows)");
    c->launches++;
    return note_err(c, sk_launch_rp<SK_LIN>(maps, p, grid, st, !(c->cfg.flags & MRP_FLAG_NO_PDL), false),
                    "module q, k, v kernel (few rows)");
}

// act[n, F] = silu(rstd * A Wg^T) * (rstd * A Wu^T) in operand form (lo rows sk_head_pad(n) rows further on).
cudaError_t sk_gate_up(Ctx *c, const __nv_bfloat16 *a, int n, int n_in, const void *w_gate, const void *w_up, int F,
                       const float *sumsq, int n_ss, __nv_bfloat16 *act, int32_t *user_status, cudaStream_t st)
{
    const TcState *s = (const TcState *)c->tc_state;
    SkParams p;
    memset(&p, 0, sizeof(p));
    p.M = n; p.d = n_in; p.F = F;
    p.status = (int32_t *)(c->ws + c->lay.status); p.user_status = user_status;
    p.units_total = F / 8; p.k_chunks = n_in / kBK; p.r_pad = sk_head_pad(n); p.w_rows = F;
    p.lo_x = p.r_pad; p.lo_xt = p.r_pad;
    p.sumsq = sumsq; p.n_ss = n_ss; p.eps = c->cfg.rms_eps; p.act = act;
    sk_finish_shape(p, 0);
    const int grid = sk_split(c, p, F / 64);
    SkMaps maps;
    memset(&maps, 0, sizeof(maps));
    if (!make_map(s, &maps.x, a, n_in, 2 * (uint64_t)p.r_pad, 2 * p.r_pad) ||
        !sk_weight_maps(s, maps, 0, w_gate, n_in, F, 8, p) || !sk_weight_maps(s, maps, 1, w_up, n_in, F, 8, p))
        return note_err(c, cudaErrorInvalidValue, "tensor map (module gate/up, few rows)");
    c->launches++;
    return note_err(c, sk_launch_rp<SK_GU>(maps, p, grid, st, !(c->cfg.flags & MRP_FLAG_NO_PDL), false),
                    "module gate/up kernel (few rows)");
}

cudaError_t sk_lm(Ctx *c, const float *logits0, const int32_t *row_index, int M, int K,
                  const mrp_draft_out &out, cudaStream_t st, bool pdl)
{
    const TcState *s = (const TcState *)c->tc_state;
    const int d = c->cfg.d, V = c->cfg.vocab, G = c->sm_count;
    SkParams p;
    sk_common(c, p, M, K, out);
    p.units_total = V / 16; p.k_chunks = d / kBK; p.r_pad = sk_lm_pad(p.n_rs);
    p.kc = (p.k_chunks % 2 == 0) ? 2 : 1;
    p.logits0 = logits0; p.row_index = row_index; p.n_rows_in = c->input_rows; p.l0_bf16 = c->l0_bf16 ? 1 : 0;
    p.partials = (Partial *)(c->ws + c->lay.partials); p.logits_out = out.logits_out;
    SkMaps maps;
    memset(&maps, 0, sizeof(maps));
    if (c->use_fp8_lm) {
        // the operand rows as e4m3 limbs, then the same kernel on the 8-bit copy of W_lm
        uint8_t *xq = (uint8_t *)(c->ws + c->lay.xq);
        float *xs = (float *)(c->ws + c->lay.x8_scale);
        cudaError_t e = note_err(c, launch_k(operand_limbs_kernel, dim3(p.n_rs), dim3(256), 0, st, pdl,
                                             (const __nv_bfloat16 *)(c->ws + c->lay.xt), c->lo_xt, d, p.r_pad, xq, xs),
                                 "operand limb kernel");
        c->launches++;
        if (e != cudaSuccess) return e;
        p.k_chunks = d / 128; p.kc = 2; p.n_parts = 4;
        p.w8_scale = (const float *)(c->ws + c->lay.w8_scale); p.x8_scale = xs;
        sk_finish_shape(p, G);
        bool ok = make_map_u8(s, &maps.x, xq, d, 4 * (uint64_t)p.r_pad, 4 * p.r_pad) &&
                  make_map_u8(s, &maps.w[0], c->ws + c->lay.w8, d, V, 128);
        static const int slot[4] = {1, 2, 4, 5};
        for (int k = 0; k < 4 && ok; ++k)
            if (p.lm_h[k] > 0) ok = make_map_u8(s, &maps.w[slot[k]], c->ws + c->lay.w8, d, V, p.lm_h[k] * 16);
        if (!ok) return note_err(c, cudaErrorInvalidValue, "tensor map (LM head, 8-bit weights)");
        c->launches++;
        return note_err(c, sk_launch_rp<SK_LM>(maps, p, G, st, pdl, out.margin != nullptr), "LM-head kernel (8-bit weights)");
    }
    sk_finish_shape(p, G);
    if (!make_map(s, &maps.x, c->ws + c->lay.xt, d, 2 * (uint64_t)p.r_pad, 2 * p.r_pad) ||
        !sk_weight_maps(s, maps, 0, c->w_lm, d, V, 16, p))
        return note_err(c, cudaErrorInvalidValue, "tensor map (LM head, few rows)");
    c->launches++;
    return note_err(c, sk_launch_rp<SK_LM>(maps, p, G, st, pdl, out.margin != nullptr), "LM-head kernel (few rows)");
}

bool fp8_lm_supported(const mrp_config &cfg)
{
    return cfg.dtype == MRP_BF16 && !(cfg.flags & (MRP_FLAG_FORCE_SIMT | MRP_FLAG_ROW_MAJOR_ONLY | MRP_FLAG_TRAINING_KL)) &&
           cfg.d % 256 == 0 && cfg.n_heads >= 1 && ((long long)cfg.n_heads + 1) * cfg.max_rows <= 32;
}

cudaError_t fp8_lm_create(Ctx *c)
{
    quantise_rows_kernel<<<c->cfg.vocab, 256>>>((const __nv_bfloat16 *)c->w_lm, c->cfg.d, (uint8_t *)(c->ws + c->lay.w8),
                                                (float *)(c->ws + c->lay.w8_scale));
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) e = cudaMemset(c->ws + c->lay.xq, 0, (size_t)4 * 32 * c->cfg.d);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    c->use_fp8_lm = (e == cudaSuccess);
    return e;
}

}  // namespace mrp
