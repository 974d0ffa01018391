// Tensor-core kernel family, row-major form (sm_100a): tcgen05.mma with TMEM accumulators, operands
// staged in shared memory by TMA (128-byte swizzle), warp-specialised: one TMA producer thread,
// one MMA issuer warp (one elected lane issues), four epilogue warps that read the accumulators back with tcgen05.ld.
// Used where there are many activation rows; tc_skinny.cu holds the few-row form.
//
// All three GEMMs of the drafting pass share one main loop and differ in the epilogue:
//   GU  gate/up projections of a head:  act = silu(rstd * Wg x) * (rstd * Wu x)          (a1)
//   DN  down projection:  h <- h + Wd act, emits the operands of the next GEMMs           (a1)
//   LM  shared LM head on the stacked residual rows h_k - h_0 of steps 1..K, fused with
//       "+ l_0" and the online softmax statistics (max, sum of exponentials, argmax,
//       runner-up); the statistics of step 0 ride on the rows of step 1               (a2, a3)
// Precision: weights are exact bf16.  Activation operands are a pair of bf16 matrices hi + lo
// (lo = bf16 of what hi lost), both multiplied by every weight tile into one accumulator, so the
// products are exact to about 2^-17.  The LM head above 128 row-steps instead takes its operand
// rounded once to fp16 against an fp16 copy of W_lm (one MMA pass; the combine then recomputes
// each row-step's top logit exactly).
// Orientation: activation rows are the MMA M dimension (128 TMEM lanes, one row per epilogue
// thread), weight rows the MMA N dimension.  A CTA is a (weight-row range, group of 128-row
// activation blocks) pair: it streams its range once per block of its group, and CTAs of the
// same range share those reads through L2.
#include <cuda_fp16.h>
#include <string.h>

#include <atomic>

#include <new>

#include "tc_common.cuh"

namespace mrp {
namespace {

constexpr int kThreads = 192;
constexpr int kATile = 128 * 128;          // bytes of a 128-row A tile
constexpr int kAccCols = 256;              // TMEM columns per accumulator buffer (two buffers)

enum { KIND_GU = 0, KIND_DN = 1, KIND_LM = 2, KIND_LIN = 3 };

struct TcParams {
    // decomposition of the weight rows (MMA N)
    int units_total;     // weight-row extent in units
    int unit_rows;       // rows per unit per B box (LM/DN 16, GU 8 of gate + 8 of up)
    int w_units;         // tile width in units
    int bn;              // MMA N = rows of the B tile
    int n_boxes;         // TMA boxes per B tile (GU 2, else 1)
    int k_chunks;        // contraction extent / 64
    int n_stages;
    // decomposition of the work over CTAs: CTA = (weight-row range, group of row blocks)
    int n_vr;            // weight-row ranges
    int n_groups;        // row-block groups; group g owns blocks g, g + n_groups, ...
    int n_rb;            // 128-row activation blocks
    int rows;            // valid activation rows (GU/DN: M; LM: K*M row-steps of steps 1..K)
    int a_row_base;      // A row coordinate of row 0 (hi part)
    int step_base;       // LM: MRP step of row 0 (1: step 0 rides on the rows of step 1; 0: it has its own rows)
    int a_part_rows;     // A row offset from the hi part to the lo part
    int M, K, V, d, F;
    int n_rs;            // (K+1)*M
    // LM
    const float *logits0;
    const int32_t *row_index;
    int n_rows_in;       // row_index entries at or above are invalid: their base logits read as zero
    int l0_bf16;         // logits0 holds bf16 values
    Partial *partials;
    float *logits_out;
    const float *teacher;        // KL variant: teacher logits [K * M, V], row-step order of steps 1..K
    KlPartial *kl_partials;      // [n_vr][K * M]
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
    __half *xt16_k;      // optional: the same rows rounded once to fp16
    float *sumsq_out;
    float *hidden_out;
    // LIN: a plain product, out[row, j] (+)= rstd(row) * acc (rstd from `sumsq` as in GU, 1 without it)
    float *lin_out;
    int lin_n_out;
    int lin_accumulate;
    // LIN over lin_nw = 3 weight matrices of the same shape sharing the activation rows (q, k, v of the module):
    // the weight-row ranges are dealt out per matrix (n_vr / 3 each), results to lin_out, lin_out1, lin_out2
    int lin_nw;
    float *lin_out1, *lin_out2;
    int32_t *status;
    int32_t *user_status;
};

// ---------------------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------------------
// F16: one fp16 A tile per stage against fp16 weights (LM head only); otherwise the bf16 hi and lo
// A tiles of a k-chunk against bf16 weights.
// PAIR: the grid is launched in clusters of two CTAs that share every MMA (cta_group::2, M = 256): CTA r of
// a pair owns row block pb + r * (number of pairs of blocks) -- with an even number K of steps stacked these are
// the same masked rows at steps k and k + K / 2, so that the pair reads each tile of their base logits from
// DRAM once -- and loads its own A tiles plus HALF of the B tile (rows r * bn / 2 ...),
// which halves the weight bytes a CTA pulls from L2 per MMA cycle and so deepens the ring.  The leader
// (rank 0) issues the MMAs; both CTAs' loads complete on the leader's full barrier; the MMA commits
// arrive on both CTAs' empty / accumulator-full barriers; both CTAs' epilogue warps arrive on the
// leader's accumulator-empty barrier.  No load is multicast: each CTA fetches its own tiles.
template <int KIND, bool MARGIN, bool F16, bool KL, bool PAIR = false>
__global__ void __launch_bounds__(kThreads, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB0,
               const __grid_constant__ CUtensorMap tmB1, const __grid_constant__ CUtensorMap tmB2, const TcParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    // a stage holds the A tile(s) of a k-chunk and one B tile (PAIR: this CTA's half of it)
    constexpr int PARTS = F16 ? 1 : 2;
    const int bn_own = PAIR ? p.bn / 2 : p.bn;           // B rows in this CTA's shared memory
    const int b_bytes = (bn_own * 128 + 1023) & ~1023;
    const int stage_bytes = PARTS * kATile + b_bytes;
    const uint32_t bars = base + (uint32_t)p.n_stages * stage_bytes;   // 8-byte aligned
    // barrier slots: full[s], empty[s], tmem_full[2], tmem_empty[2]
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (p.n_stages + s); };
    auto tfull_bar = [&](int a) { return bars + 8u * (2 * p.n_stages + a); };
    auto tempty_bar = [&](int a) { return bars + 8u * (2 * p.n_stages + 2 + a); };
    uint8_t *gen_base = smem_raw + (base - smem_u32(smem_raw));
    uint32_t *tmem_holder = reinterpret_cast<uint32_t *>(gen_base + (size_t)p.n_stages * stage_bytes + 8 * (2 * p.n_stages + 4));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_holder + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // PAIR: `cta` numbers the pair, `rank` the CTA in it; a pair walks PAIRS of row blocks (p.n_rb counts pairs,
    // row block of this CTA = pair-block + rank * p.n_rb)
    const int rank = PAIR ? (int)cluster_ctarank() : 0;
    const int cta = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
    const int vr = cta % p.n_vr, grp = cta / p.n_vr;
    // (LIN over three matrices: `which` of them this CTA works on, and its range among that matrix's n_vr / 3)
    const int n_vr_w = (KIND == KIND_LIN && p.lin_nw == 3) ? p.n_vr / 3 : p.n_vr;
    const int which = (KIND == KIND_LIN && p.lin_nw == 3) ? vr / n_vr_w : 0;
    const int vr_w = vr - which * n_vr_w;
    const CUtensorMap *tmB = which == 0 ? &tmB0 : which == 1 ? &tmB1 : &tmB2;
    float *lin_dst = which == 0 ? p.lin_out : which == 1 ? p.lin_out1 : p.lin_out2;
    const int u0 = (int)((long long)vr_w * p.units_total / n_vr_w);
    const int u1 = (int)((long long)(vr_w + 1) * p.units_total / n_vr_w);
    const int n_t = (u1 - u0 + p.w_units - 1) / p.w_units;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.n_stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), PAIR ? 8 : 4); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        prefetch_tmap(&tmA);
        prefetch_tmap(KIND == KIND_LIN ? tmB : &tmB0);
        if (KIND == KIND_GU) prefetch_tmap(&tmB1);
    }
    if (warp == 1) {
        if (PAIR) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32(tmem_holder)), "r"(2u * kAccCols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32(tmem_holder)), "r"(2u * kAccCols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync_all();       // both CTAs' barriers exist before either signals the other's
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;
    // launched behind its predecessor with programmatic dependent launch: everything above overlaps
    // the predecessor's tail; the roles that touch its outputs wait for it first
    pdl_trigger();

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            // PAIR: both CTAs' loads are counted by the leader's barrier, which its producer arms for both
            const uint32_t tx = (uint32_t)(PARTS * kATile + bn_own * 128) * (PAIR ? 2u : 1u);
            const int box_rows = p.bn / p.n_boxes;
            // the CTA's work as one sequence of ring steps: row blocks mb = grp, grp + n_groups, ...,
            // for each its n_t weight tiles, for each tile the k-chunks
            auto advance = [&](int &mb_, int &t_, int &kk_) {
                if (++kk_ == p.k_chunks) { kk_ = 0; if (++t_ == n_t) { t_ = 0; mb_ += p.n_groups; } }
            };
            auto load_b = [&](int t_, int kk_, int s_) {
                const int n0 = (u0 + t_ * p.w_units) * p.unit_rows;
                const uint32_t sb = base + (uint32_t)s_ * stage_bytes + PARTS * kATile;
                if (PAIR) {
                    // this CTA's half of the B tile: rows [rank * bn / 2, ...) of a one-box tile; of a gate/up tile
                    // the gate rows (leader) or the up rows (peer), so that the columns stay [gate | up]
                    if (KIND == KIND_GU) tma_load_2d_pair(sb, rank ? &tmB1 : &tmB0, kk_ * kBK, n0, full_bar(s_));
                    else tma_load_2d_pair(sb, KIND == KIND_LIN ? tmB : &tmB0, kk_ * kBK, n0 + rank * bn_own, full_bar(s_));
                } else {
                    tma_load_2d(sb, KIND == KIND_LIN ? tmB : &tmB0, kk_ * kBK, n0, full_bar(s_));
                    if (KIND == KIND_GU) tma_load_2d(sb + box_rows * 128, &tmB1, kk_ * kBK, n0, full_bar(s_));
                }
            };
            auto load_a = [&](int mb_, int kk_, int s_) {
                const uint32_t sa = base + (uint32_t)s_ * stage_bytes;
                const int row0 = p.a_row_base + (PAIR ? mb_ + rank * p.n_rb : mb_) * 128;
                if (PAIR) {
                    tma_load_2d_pair(sa, &tmA, kk_ * kBK, row0, full_bar(s_));
                    if (!F16) tma_load_2d_pair(sa + kATile, &tmA, kk_ * kBK, p.a_part_rows + row0, full_bar(s_));
                } else {
                    tma_load_2d(sa, &tmA, kk_ * kBK, row0, full_bar(s_));
                    if (!F16) tma_load_2d(sa + kATile, &tmA, kk_ * kBK, p.a_part_rows + row0, full_bar(s_));
                }
            };
            auto arm = [&](int s_) { if (!PAIR || rank == 0) mbar_expect_tx(full_bar(s_), tx); };
            const int my_blocks = grp < p.n_rb ? (p.n_rb - 1 - grp) / p.n_groups + 1 : 0;
            const long long total_it = (long long)my_blocks * n_t * p.k_chunks;
            const int pre = (int)(total_it < p.n_stages ? total_it : p.n_stages);
            // the weight tiles depend on nothing: the ring is filled with them while the previous
            // kernel of the stream drains; only the activation tiles wait for it
            int mb = grp, t = 0, kk = 0;
            for (int it = 0; it < pre; ++it) {
                arm(it);
                load_b(t, kk, it);
                advance(mb, t, kk);
            }
            pdl_wait();
            {
                int mb2 = grp, t2 = 0, kk2 = 0;
                for (int it = 0; it < pre; ++it) { load_a(mb2, kk2, it); advance(mb2, t2, kk2); }
            }
            int s = 0;
            uint32_t ph = 1;              // the ring has been filled once
            for (long long it = pre; it < total_it; ++it) {
                if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, p)) break;
                arm(s);
                load_a(mb, kk, s);
                load_b(t, kk, s);
                advance(mb, t, kk);
                if (++s == p.n_stages) { s = 0; ph ^= 1u; }
            }
            if (PAIR) {
                // the leader's last commits also arrive here: let them land before this CTA may leave
                for (int i = 0; i < pre && !*abort_flag; ++i) {
                    if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, p)) break;
                    if (++s == p.n_stages) { s = 0; ph ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        // The whole warp walks the loop (all values are warp-uniform); the elected lane issues.
        const uint32_t idesc = PAIR ? make_idesc_pair(p.bn, F16) : F16 ? make_idesc_f16(p.bn) : make_idesc(p.bn);
        const uint32_t tm = __shfl_sync(0xffffffffu, tmem_base, 0);
        int s = 0, acc = 0;
        uint32_t ph = 0, acc_ph = 0;
        bool ok = true;
        // PAIR: the leader's warp issues for both CTAs; the peer's warp only holds the TMEM allocation
        for (int mb = grp; mb < p.n_rb && ok && rank == 0; mb += p.n_groups) {
            for (int t = 0; t < n_t && ok; ++t) {
                ok = __all_sync(0xffffffffu, mbar_wait(tempty_bar(acc), acc_ph ^ 1u, abort_flag, p));
                if (!ok) break;
                tc_fence_after();
                const uint32_t dt = tm + (uint32_t)(acc * kAccCols);
                for (int kk = 0; kk < p.k_chunks; ++kk) {
                    const uint32_t sa = base + (uint32_t)s * stage_bytes;
                    const uint64_t db = make_smem_desc(sa + PARTS * kATile);
                    const uint32_t later = kk > 0 ? 1u : 0u;
                    ok = __all_sync(0xffffffffu, mbar_wait(full_bar(s), ph, abort_flag, p));
                    if (!ok) break;
                    tc_fence_after();
                    if (elect_one()) {
#pragma unroll
                        for (int a = 0; a < PARTS; ++a) {
                            const uint64_t da = make_smem_desc(sa + a * kATile);
#pragma unroll
                            for (int k4 = 0; k4 < kBK / 16; ++k4) {
                                if (PAIR) umma_bf16_pair(dt, da + 2u * k4, db + 2u * k4, idesc, (k4 > 0 || a > 0) ? 1u : later);
                                else umma_bf16(dt, da + 2u * k4, db + 2u * k4, idesc, (k4 > 0 || a > 0) ? 1u : later);
                            }
                        }
                        if (PAIR) umma_commit_pair(empty_bar(s));
                        else umma_commit(empty_bar(s));
                    }
                    __syncwarp();
                    if (++s == p.n_stages) { s = 0; ph ^= 1u; }
                }
                if (!ok) break;
                if (elect_one()) {
                    if (PAIR) umma_commit_pair(tfull_bar(acc));
                    else umma_commit(tfull_bar(acc));
                }
                __syncwarp();
                acc ^= 1;
                if (acc == 0) acc_ph ^= 1u;
            }
        }
    } else {
        // ---------------- epilogue warps (TMEM lane quadrant = warp % 4) ----------------
        pdl_wait();
        const int q = warp & 3;
        const int rl = q * 32 + lane;
        const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
        int acc = 0;
        uint32_t acc_ph = 0;
        bool ok = true;
        for (int mb = grp; mb < p.n_rb && ok; mb += p.n_groups) {
            // ---- per-block state: this thread's activation row ----
            const int r = (PAIR ? mb + rank * p.n_rb : mb) * 128 + rl;
            const bool valid = r < p.rows;
            RowStat st, st0;       // LM: statistics of the row's own step, and of step 0 (rows of step 1 only)
            KlStat kst;            // LM, KL variant: the row-step's share of the training objective
            const float *tp = nullptr;
            bool first_step = false;
            const float *l0p = nullptr;
            int k_of_row = 0, m_of_row = r;
            float rstd = 0.f, ssq = 0.f;
            if (KIND == KIND_LM) {
                st.init();
                st0.init();
                if (valid) {
                    k_of_row = r / p.M + p.step_base;
                    m_of_row = r - (k_of_row - p.step_base) * p.M;
                    first_step = (k_of_row == 1 && p.step_base == 1);
                    const int idx = p.row_index ? p.row_index[m_of_row] : m_of_row;
                    // (for bf16 base logits l0p is kept in units of two bytes: see the load below)
                    if (p.logits0 && (!p.row_index || row_ok(idx, p.n_rows_in)))
                        l0p = p.l0_bf16 ? reinterpret_cast<const float *>(reinterpret_cast<const __nv_bfloat16 *>(p.logits0) +
                                                                           (size_t)idx * (size_t)p.V)
                                        : p.logits0 + (size_t)idx * (size_t)p.V;
                    if (KL) {
                        kst.init();
                        tp = p.teacher + ((size_t)(k_of_row - 1) * p.M + m_of_row) * (size_t)p.V;   // step_base is 1 here
                    }
                }
            } else if ((KIND == KIND_GU || (KIND == KIND_LIN && p.sumsq)) && valid) {
                float s = 0.f;
                for (int i = 0; i < p.n_ss; ++i) s += p.sumsq[(size_t)i * p.M + m_of_row];
                rstd = rsqrtf(s / (float)p.d + p.eps);
            }
            for (int t = 0; t < n_t && ok; ++t) {
                ok = __all_sync(0xffffffffu, mbar_wait(tfull_bar(acc), acc_ph, abort_flag, p));
                if (!ok) break;
                tc_fence_after();
                const int ut = u0 + t * p.w_units;
                const int units_here = min(p.w_units, u1 - ut);
                const uint32_t tacc = lane_addr + (uint32_t)(acc * kAccCols);
                if (KIND == KIND_LM) {
                    const int v_tile = ut * 16;
                    for (int c = 0; c < units_here; ++c) {
                        const int v = v_tile + c * 16;
                        float l0[16], a[16];
                        if (valid && p.logits0) {
                            if (l0p) {
                                if (p.l0_bf16) load16_bf16(reinterpret_cast<const __nv_bfloat16 *>(l0p) + v, l0);
                                else load16(l0p + v, l0);
                            } else {          // the caller's row index was out of range: an all-zero logit row
#pragma unroll
                                for (int j = 0; j < 16; ++j) l0[j] = 0.f;
                            }
                        }
                        float tch[16];
                        if (KL && valid) load16(tp + v, tch);
                        tmem_ld16(tacc + c * 16, a);
                        if (valid) {
                            if (p.logits0) {
                                if (first_step) st0.template update<MARGIN>(l0, v);
#pragma unroll
                                for (int j = 0; j < 16; ++j) a[j] += l0[j];
                            }
                            st.template update<MARGIN>(a, v);
                            if (KL) kst.update(tch, a);
                            if (p.logits_out && k_of_row >= 1)
                                store16(p.logits_out + ((size_t)(k_of_row - 1) * p.M + m_of_row) * p.V + v, a);
                        }
                    }
                } else if (KIND == KIND_GU) {
                    const int ng = p.bn >> 1;
                    const int f_tile = ut * 8;
                    for (int c = 0; c < units_here; ++c) {
                        float g[8], u[8];
                        tmem_ld8(tacc + c * 8, g);
                        tmem_ld8(tacc + ng + c * 8, u);
                        if (valid) {
                            float av[8];
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                const float gj = g[j] * rstd;
                                av[j] = gj / (1.f + __expf(-gj)) * (u[j] * rstd);
                            }
                            store_split<8>(p.act + (size_t)m_of_row * p.F + f_tile + c * 8, (size_t)p.M * p.F, av);
                        }
                    }
                } else if (KIND == KIND_LIN) {
                    const int j_tile = ut * 16;
                    for (int c = 0; c < units_here; ++c) {
                        float a[16];
                        tmem_ld16(tacc + c * 16, a);
                        if (valid) {
                            const size_t o = (size_t)m_of_row * p.lin_n_out + j_tile + c * 16;
                            if (p.sumsq) {
#pragma unroll
                                for (int j = 0; j < 16; ++j) a[j] *= rstd;
                            }
                            if (p.lin_accumulate) {
                                float z[16];
                                load16_rw(lin_dst + o, z);
#pragma unroll
                                for (int j = 0; j < 16; ++j) a[j] += z[j];
                            }
                            store16(lin_dst + o, a);
                            if (p.xg_next) {
                                // the next product's operand rows, out * gamma_next as bf16 hi + lo, and this CTA's
                                // share of the row's sum of squares (its RMSNorm)
                                const __nv_bfloat16 *gm = p.gamma_next + j_tile + c * 16;
                                float x[16];
#pragma unroll
                                for (int j = 0; j < 16; ++j) {
                                    ssq = fmaf(a[j], a[j], ssq);
                                    x[j] = a[j] * __bfloat162float(gm[j]);
                                }
                                store_split<16>(p.xg_next + o, (size_t)p.M * p.lin_n_out, x);
                            }
                        }
                    }
                } else {
                    const int j_tile = ut * 16;
                    for (int c = 0; c < units_here; ++c) {
                        float a[16];
                        tmem_ld16(tacc + c * 16, a);
                        if (valid) {
                            const size_t o = (size_t)m_of_row * p.d + j_tile + c * 16;
                            float hc[16], h0[16];
                            load16_rw(p.hcur + o, hc);
                            load16(p.h0f + o, h0);
#pragma unroll
                            for (int j = 0; j < 16; ++j) { hc[j] += a[j]; ssq = fmaf(hc[j], hc[j], ssq); }
                            store16(p.hcur + o, hc);
                            if (p.hidden_out) store16(p.hidden_out + o, hc);
#pragma unroll
                            for (int j = 0; j < 16; ++j) h0[j] = hc[j] - h0[j];
                            store_split<16>(p.xt_k + o, (size_t)p.n_rs * p.d, h0);
                            if (p.xt16_k) {
                                __half2 hh[8];
#pragma unroll
                                for (int j = 0; j < 8; ++j) hh[j] = __floats2half2_rn(h0[2 * j], h0[2 * j + 1]);
                                uint4 *dst = reinterpret_cast<uint4 *>(p.xt16_k + o);
                                dst[0] = *reinterpret_cast<uint4 *>(&hh[0]);
                                dst[1] = *reinterpret_cast<uint4 *>(&hh[4]);
                            }
                            if (p.xg_next) {
                                const __nv_bfloat16 *gm = p.gamma_next + j_tile + c * 16;
#pragma unroll
                                for (int j = 0; j < 16; ++j) hc[j] *= __bfloat162float(gm[j]);
                                store_split<16>(p.xg_next + o, (size_t)p.M * p.d, hc);
                            }
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    if (PAIR) mbar_arrive_leader(tempty_bar(acc));
                    else mbar_arrive(tempty_bar(acc));
                }
                acc ^= 1;
                if (acc == 0) acc_ph ^= 1u;
            }
            // ---- per-block results ----
            if (ok && valid) {
                if (KIND == KIND_LM) {
                    p.partials[(size_t)vr * p.n_rs + (size_t)k_of_row * p.M + m_of_row] = st.partial();
                    if (first_step) p.partials[(size_t)vr * p.n_rs + m_of_row] = st0.partial();
                    if (KL)
                        p.kl_partials[(size_t)vr * ((size_t)p.K * p.M) + (size_t)(k_of_row - 1) * p.M + m_of_row] = kst.partial();
                } else if (KIND == KIND_DN) {
                    p.sumsq_out[(size_t)vr * p.M + m_of_row] = ssq;
                } else if (KIND == KIND_LIN && p.xg_next) {
                    p.sumsq_out[(size_t)vr * p.M + m_of_row] = ssq;
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
    // PAIR: neither CTA leaves, nor frees the shared allocation, while the other may still signal its barriers
    if (PAIR) cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        if (PAIR)
            asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(2u * kAccCols) : "memory");
        else
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(2u * kAccCols) : "memory");
    }
}

// Gather masked rows: fp32 copies of h_0, the first head's operand bf16(h_0 * gamma_1), the
// row sums of squares, and the zero rows that stand for step 0 in the stacked LM-head operand.
// Without base logits (from_hidden) the LM-head operand of step k is n_0 + (h_k - h_0), so that
// the pass itself yields l_k = W_lm n_0 + W_lm (h_k - h_0): the step-0 rows hold n_0 = h_0, or
// RMSNorm(h_0) * final_gamma, and h0f holds h_0 - n_0, which is what the down-projection
// epilogues subtract from h_k.
__global__ void tc_prep_kernel(const __nv_bfloat16 *__restrict__ hidden, const int32_t *__restrict__ row_index,
                               int d, int lo_x, int lo_xt, const __nv_bfloat16 *__restrict__ gamma1,
                               float *__restrict__ h0f, float *__restrict__ hcur, __nv_bfloat16 *__restrict__ xg,
                               __nv_bfloat16 *__restrict__ xt0, float *__restrict__ sumsq,
                               int32_t *__restrict__ counters, int n_counters,
                               unsigned long long *__restrict__ ssq_fix, int from_hidden,
                               const __nv_bfloat16 *__restrict__ final_gamma, float eps, __half *__restrict__ xt16_0,
                               int n_rows_in, int32_t *__restrict__ status, int32_t *__restrict__ user_status)
{
    pdl_trigger();
    pdl_wait();
    // arrival counters of the few-row head kernels start every pass at zero
    if (blockIdx.x == 0)
        for (int i = threadIdx.x; i < n_counters; i += blockDim.x) counters[i] = 0;
    __shared__ float red[8];
    __shared__ float total_s;
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
        const float v = bad ? 0.f : __bfloat162float(hidden[row * d + j]);
        const size_t o = (size_t)m * d + j;
        if (!from_hidden) h0f[o] = v;
        hcur[o] = v;
        if (gamma1) {
            const float x = v * __bfloat162float(gamma1[j]);
            const __nv_bfloat16 hi = __float2bfloat16_rn(x);
            xg[o] = hi;
            xg[(size_t)lo_x * d + o] = __float2bfloat16_rn(x - __bfloat162float(hi));
        }
        if (!from_hidden) {
            xt0[o] = __float2bfloat16(0.f);
            xt0[(size_t)lo_xt * d + o] = __float2bfloat16(0.f);
        }
        ss = fmaf(v, v, ss);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    if (threadIdx.x == 0) {
        float t = 0.f;
        for (int i = 0; i < (int)(blockDim.x >> 5); ++i) t += red[i];
        sumsq[m] = t;
        if (m < 128) {
            // the chain kernel keeps sums of squares in 2^-24 fixed point (integer adds commute)
            ssq_fix[m] = (unsigned long long)__double2ll_rn((double)t * 16777216.0);
            for (int k = 1; k < 5; ++k) ssq_fix[k * 128 + m] = 0ull;
        }
        total_s = t;
    }
    if (from_hidden) {
        __syncthreads();
        const float rstd0 = final_gamma ? rsqrtf(total_s / (float)d + eps) : 1.f;
        for (int j = threadIdx.x; j < d; j += blockDim.x) {
            const float v = bad ? 0.f : __bfloat162float(hidden[row * d + j]);
            const float n0 = final_gamma ? v * rstd0 * __bfloat162float(final_gamma[j]) : v;
            const size_t o = (size_t)m * d + j;
            h0f[o] = v - n0;
            const __nv_bfloat16 hi = __float2bfloat16_rn(n0);
            xt0[o] = hi;
            xt0[(size_t)lo_xt * d + o] = __float2bfloat16_rn(n0 - __bfloat162float(hi));
            if (xt16_0) xt16_0[o] = __float2half_rn(n0);
        }
    }
}

// fp16 copy of a bf16 matrix.  bf16 values inside fp16's normal range convert exactly; smaller
// ones round to fp16 subnormals (absolute error <= 2^-25); flag[0] is set if a finite value
// overflows fp16 or a value is not finite, which rules the copy out.
__global__ void to_half_kernel(const __nv_bfloat16 *__restrict__ src, __half *__restrict__ dst, size_t n,
                               int32_t *__restrict__ flag)
{
    bool bad = false;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const float v = __bfloat162float(src[i]);
        const __half h = __float2half_rn(v);
        bad |= !isfinite(__half2float(h));
        dst[i] = h;
    }
    if (bad) atomicOr(flag, 1);
}

// One thread waits for an mbarrier nobody completes: the bounded wait must give up and report.
struct SelfTestParams { int32_t *status, *user_status; };
__global__ void selftest_timeout_kernel(SelfTestParams p)
{
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_wait(smem_u32(&bar), 0u, &abort_flag, p);
    }
}

// ---------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------
// Tile width (in units, at most w_max) for CTAs owning up to `maxunits` units.  An MMA costs
// about the same whatever its N, so the tile count is kept minimal first; among the widths that
// reach it the narrowest wastes the fewest rows beyond the range.
int choose_tile_units(int maxunits, int w_max)
{
    const int t_min = (maxunits + w_max - 1) / w_max;
    return (maxunits + t_min - 1) / t_min;
}

// Split of the work over `G` CTAs: n_groups row-block groups times G / n_groups weight-row
// ranges, chosen for the shortest longest CTA (in 16-unit tiles), the fewest passes on ties.
int choose_groups(int n_rb, int units_total, int G)
{
    int best_g = 1;
    long long best_cost = -1;
    for (int g = 1; g <= n_rb && g <= G; ++g) {
        const int nv = G / g;
        const int passes = (n_rb + g - 1) / g;
        const int units = (units_total + nv - 1) / nv;
        const long long cost = (long long)passes * ((units + 15) / 16);
        if (best_cost < 0 || cost <= best_cost) { best_cost = cost; best_g = g; }
    }
    return best_g;
}

// CTA pairs need an even number of SMs, all of which clusters of two can occupy at once (otherwise the
// grid would run in waves), and can be switched off per context.
bool pair_ok(const Ctx *c)
{
    return !(c->cfg.flags & MRP_FLAG_NO_CTA_PAIRS) && (c->sm_count % 2 == 0);
}

void finish_shape(TcParams &p, int n_vr, int parts = 2, bool pair = false)
{
    p.n_vr = n_vr;
    const int maxunits = (p.units_total + n_vr - 1) / n_vr;
    const int bn_max = kAccCols;
    const int rows_per_unit = p.unit_rows * p.n_boxes;
    int w_max = bn_max / rows_per_unit;
    if (w_max > 256 / rows_per_unit) w_max = 256 / rows_per_unit;
    if (w_max < 1) w_max = 1;
    p.w_units = choose_tile_units(maxunits < 1 ? 1 : maxunits, w_max);
    p.bn = p.w_units * rows_per_unit;
    const int b_bytes = ((pair ? p.bn / 2 : p.bn) * 128 + 1023) & ~1023;
    const int stage = parts * kATile + b_bytes;
    int ns = (kSmemBudget - 1024 - 512) / stage;
    if (ns > 12) ns = 12;
    p.n_stages = ns;
}

size_t smem_bytes(const TcParams &p, int parts, bool pair)
{
    const int b_bytes = ((pair ? p.bn / 2 : p.bn) * 128 + 1023) & ~1023;
    return (size_t)p.n_stages * (parts * kATile + b_bytes) + 1024 + 8 * (2 * p.n_stages + 4) + 16;
}

// PAIR: `grid` counts CTAs (two per pair); the launch carries the cluster shape (2, 1, 1).
template <int KIND, bool MARGIN, bool F16 = false, bool KL = false, bool PAIR = false>
cudaError_t launch_tc(const CUtensorMap &a, const CUtensorMap &b0, const CUtensorMap &b1, const TcParams &p,
                      int grid, cudaStream_t st, bool pdl, const CUtensorMap *b2_opt = nullptr)
{
    const CUtensorMap &b2 = b2_opt ? *b2_opt : b1;
    auto kern = tc_gemm_kernel<KIND, MARGIN, F16, KL, PAIR>;
    const size_t smem = smem_bytes(p, F16 ? 1 : 2, PAIR);
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
    if (PAIR) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(grid);
        cfg.blockDim = dim3(kThreads);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = st;
        cudaLaunchAttribute at[2];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[1].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = at;
        cfg.numAttrs = pdl ? 2 : 1;
        return cudaLaunchKernelEx(&cfg, kern, a, b0, b1, b2, p);
    }
    return launch_k(kern, dim3(grid), dim3(kThreads), smem, st, pdl, a, b0, b1, b2, p);
}

}  // namespace

cudaError_t tc_selftest_timeout(Ctx *c, int32_t *user_status, cudaStream_t st)
{
    SelfTestParams p;
    p.status = (int32_t *)(c->ws + c->lay.status);
    p.user_status = user_status;
    selftest_timeout_kernel<<<1, 32, 0, st>>>(p);
    return cudaGetLastError();
}

bool tc_supported(const mrp_config &cfg, const mrp_head_weights *heads, const void *w_lm)
{
    if (cfg.dtype != MRP_BF16) return false;
    if (cfg.d % 64 || cfg.d_ff % 64 || cfg.vocab % 16) return false;
    if ((uintptr_t)w_lm & 15u) return false;
    for (int k = 0; k < cfg.n_heads; ++k)
        if (((uintptr_t)heads[k].rms_gamma & 1u) || ((uintptr_t)heads[k].w_gate & 15u) ||
            ((uintptr_t)heads[k].w_up & 15u) || ((uintptr_t)heads[k].w_down & 15u))
            return false;
    return true;
}

cudaError_t tc_create(Ctx *c)
{
    TcState *s = new (std::nothrow) TcState;
    if (!s) return cudaErrorMemoryAllocation;
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn) {
        delete s;
        return e != cudaSuccess ? e : cudaErrorNotSupported;
    }
    s->encode = (EncodeTiledFn)fn;
    c->tc_state = s;
    c->use_f16_lm = false;
    if (c->lay.has_f16) {
        // one-time fp16 copy of the LM head for the tensor-core-bound regime
        int32_t *flag = (int32_t *)(c->ws + c->lay.status) + 8;
        e = cudaMemset(flag, 0, sizeof(int32_t));
        if (e != cudaSuccess) return e;
        to_half_kernel<<<c->sm_count * 8, 256>>>((const __nv_bfloat16 *)c->w_lm, (__half *)(c->ws + c->lay.w16),
                                                 (size_t)c->cfg.vocab * c->cfg.d, flag);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        int32_t bad = 1;
        e = cudaMemcpy(&bad, flag, sizeof(bad), cudaMemcpyDeviceToHost);
        if (e != cudaSuccess) return e;
        c->use_f16_lm = (bad == 0);
    }
    return cudaSuccess;
}

void tc_destroy(Ctx *c)
{
    delete (TcState *)c->tc_state;
    c->tc_state = nullptr;
}

TcPlan tc_plan(Ctx *c, int M, int K, const mrp_draft_out &out, cudaStream_t st, bool want_chain)
{
    TcPlan pl;
    pl.n_rs = (K + 1) * M;
    pl.pdl = !(c->cfg.flags & MRP_FLAG_NO_PDL);
    pl.few_rows = sk_head_rows_ok(M) && sk_heads_ok(c->cfg) && !(c->cfg.flags & MRP_FLAG_ROW_MAJOR_ONLY);
    // the KL objective lives in the row-major LM-head kernel, on exact operands
    pl.with_kl = c->teacher != nullptr;
    pl.lm_few = sk_rows_ok(pl.n_rs) && !(c->cfg.flags & MRP_FLAG_ROW_MAJOR_ONLY) && !pl.with_kl;
    pl.f16_lm = c->use_f16_lm && pl.n_rs >= kF16MinRowSteps && !pl.lm_few && !pl.with_kl;
    pl.chain = want_chain && !(c->cfg.flags & (MRP_FLAG_ROW_MAJOR_ONLY | MRP_FLAG_NO_CHAIN)) && sk_heads_ok(c->cfg) &&
               sk_chain(c, M, K, out, st, pl.f16_lm, true) == cudaSuccess;
    c->lo_x = (pl.few_rows || pl.chain) ? sk_head_pad(M) : M;
    c->lo_xt = pl.lm_few ? sk_lm_pad(pl.n_rs) : pl.n_rs;
    return pl;
}

// The LM head on the stacked operand rows already in the workspace (xt, and xt16 in fp16 mode), the
// combine and the optional per-token probability: everything of a drafting pass behind the head chain.
cudaError_t tc_lm_tail(Ctx *c, const TcPlan &pl, const float *logits0, const int32_t *row_index, int M, int K,
                              const mrp_draft_out &out, cudaStream_t st)
{
    const TcState *s = (const TcState *)c->tc_state;
    const int d = c->cfg.d, F = c->cfg.d_ff, V = c->cfg.vocab, G = c->sm_count;
    __nv_bfloat16 *xt = (__nv_bfloat16 *)(c->ws + c->lay.xt);
    Partial *partials = (Partial *)(c->ws + c->lay.partials);
    int32_t *status = (int32_t *)(c->ws + c->lay.status);
    const int n_rs = pl.n_rs;
    const bool pdl = pl.pdl, lm_few = pl.lm_few, f16_lm = pl.f16_lm, with_kl = pl.with_kl;
    cudaError_t e;
    prof_mark(c, 1, st);
    e = note_err(c, wait_logits0(c, st), "wait for the base logits");
    if (e != cudaSuccess) return e;
    int n_slices = G;
    if (lm_few) {
        e = sk_lm(c, logits0, row_index, M, K, out, st, pdl);
        if (e != cudaSuccess) return e;
    } else {
        CUtensorMap mA, mB;
        TcParams p;
        memset(&p, 0, sizeof(p));
        // Row-steps of steps 1..K in 128-row blocks; CTA = (vocabulary range, group of row blocks).
        // Pick the split with the shortest longest CTA (in tiles), the fewest passes on ties.
        // (with the base logits computed in the pass, step 0 has rows of its own)
        const int step_base = c->from_hidden ? 0 : 1;
        const int rows = (K + 1 - step_base) * M, n_rb = (rows + 127) / 128, U = V / 16;
        // Two row blocks or more: CTA pairs, each MMA covering two row blocks (the kernel then counts pairs of
        // row blocks and pairs of CTAs); needs an even SM count the device can fill with clusters of two.
        const bool pair = pair_ok(c) && n_rb >= 2 && n_rb % 2 == 0 && !with_kl;
        const int n_cta = pair ? G / 2 : G, n_blk = pair ? (n_rb + 1) / 2 : n_rb;
        const int best_g = choose_groups(n_blk, U, n_cta);
        p.n_groups = best_g;
        n_slices = n_cta / best_g;
        p.n_rb = n_blk; p.rows = rows;
        p.units_total = U; p.unit_rows = 16; p.n_boxes = 1; p.k_chunks = d / kBK;
        p.a_row_base = step_base * M; p.a_part_rows = n_rs; p.step_base = step_base;
        p.M = M; p.K = K; p.V = V; p.d = d; p.F = F; p.n_rs = n_rs;
        p.logits0 = logits0; p.row_index = row_index; p.partials = partials; p.logits_out = out.logits_out;
        p.n_rows_in = c->input_rows; p.l0_bf16 = c->l0_bf16 ? 1 : 0;
        p.teacher = c->teacher; p.kl_partials = (KlPartial *)(c->ws + c->lay.kl_partials);
        p.status = status; p.user_status = out.status;
        finish_shape(p, n_slices, f16_lm ? 1 : 2, pair);
        const int grid = p.n_groups * p.n_vr * (pair ? 2 : 1);
        const int b_box = pair ? p.bn / 2 : p.bn;
        if (f16_lm) {
            // 16-bit elements either way: the bf16 tensor-map type only moves the bytes
            p.a_row_base = 0;
            if (!make_map(s, &mA, c->ws + c->lay.xt16, d, (uint64_t)rows, 128) ||
                !make_map(s, &mB, c->ws + c->lay.w16, d, V, b_box))
                return note_err(c, cudaErrorInvalidValue, "tensor map (LM head, fp16)");
            if (pair)
                e = note_err(c, out.margin ? launch_tc<KIND_LM, true, true, false, true>(mA, mB, mB, p, grid, st, pdl)
                                           : launch_tc<KIND_LM, false, true, false, true>(mA, mB, mB, p, grid, st, pdl),
                             "LM-head kernel (fp16 operands, CTA pairs)");
            else
                e = note_err(c, out.margin ? launch_tc<KIND_LM, true, true>(mA, mB, mB, p, grid, st, pdl)
                                           : launch_tc<KIND_LM, false, true>(mA, mB, mB, p, grid, st, pdl),
                             "LM-head kernel (fp16 operands)");
        } else {
            if (!make_map(s, &mA, xt, d, 2 * (uint64_t)n_rs, 128) || !make_map(s, &mB, c->w_lm, d, V, b_box))
                return note_err(c, cudaErrorInvalidValue, "tensor map (LM head)");
            if (pair)
                e = note_err(c, out.margin ? launch_tc<KIND_LM, true, false, false, true>(mA, mB, mB, p, grid, st, pdl)
                                           : launch_tc<KIND_LM, false, false, false, true>(mA, mB, mB, p, grid, st, pdl),
                             "LM-head kernel (CTA pairs)");
            else if (with_kl)
                e = note_err(c, out.margin ? launch_tc<KIND_LM, true, false, true>(mA, mB, mB, p, grid, st, pdl)
                                           : launch_tc<KIND_LM, false, false, true>(mA, mB, mB, p, grid, st, pdl),
                             "LM-head kernel (KL objective)");
            else
                e = note_err(c, out.margin ? launch_tc<KIND_LM, true>(mA, mB, mB, p, grid, st, pdl)
                                           : launch_tc<KIND_LM, false>(mA, mB, mB, p, grid, st, pdl), "LM-head kernel");
        }
        c->launches++;
        if (e != cudaSuccess) return e;
    }
    prof_mark(c, 2, st);
    TopFix fix;
    memset(&fix, 0, sizeof(fix));
    // every call: the size of the operand rows against the accuracy range; fp16 mode: the exact top logit
    fix.xt = xt; fix.logits0 = logits0; fix.row_index = row_index;
    fix.d = d; fix.V = V; fix.M = M; fix.n_rs = n_rs; fix.n_rows_in = c->input_rows; fix.l0_bf16 = c->l0_bf16 ? 1 : 0;
    fix.range_limit = MRP_RANGE_LIMIT;
    if (f16_lm) fix.w = (const __nv_bfloat16 *)c->w_lm;
    e = launch_combine(c, partials, n_slices, (K + 1) * M, out, status, st, &fix, M);
    prof_mark(c, 3, st);
    if (e != cudaSuccess) return e;
    FirstTok ft;
    memset(&ft, 0, sizeof(ft));
    ft.w = c->w_lm; ft.w_bf16 = 1; ft.logits0 = logits0; ft.row_index = row_index; ft.n_rows_in = c->input_rows;
    ft.l0_bf16 = c->l0_bf16 ? 1 : 0;
    if (c->use_fp8_lm) { ft.w = c->ws + c->lay.w8; ft.w8_scale = (const float *)(c->ws + c->lay.w8_scale); }
    ft.x = xt; ft.x_bf16 = 1; ft.lo_rows = c->lo_xt; ft.M = M; ft.K = K; ft.d = d; ft.V = V;
    return launch_first_token_prob(c, ft, out, st);
}
// out[n, n_out] (+)= rstd(row) * (A W^T): A = bf16 hi rows [n, n_in] with the lo rows n rows further on, W bf16
// [n_out, n_in]; rstd(row) = rsqrt(sumsq[row] / n_in + eps) where sumsq is given, else 1.  n_in % 64 == 0,
// n_out % 16 == 0, 16-byte aligned pointers.
// With xg_next: also writes the rows of out * gamma_next as the next product's bf16 hi + lo operand (lo rows n rows
// further on) and per-CTA partial sums of squares of out to sumsq_out[*n_ss_out, n] (the next RMSNorm).
cudaError_t tc_linear(Ctx *c, const __nv_bfloat16 *a, int n, int n_in, const void *w, int n_out, const float *sumsq,
                      int n_ss, float *out, bool accumulate, int32_t *user_status, cudaStream_t st, const void *gamma_next,
                      __nv_bfloat16 *xg_next, float *sumsq_out, int *n_ss_out)
{
    const TcState *s = (const TcState *)c->tc_state;
    const int G = c->sm_count, n_mb = (n + 127) / 128;
    CUtensorMap mA, mB;
    TcParams p;
    memset(&p, 0, sizeof(p));
    p.units_total = n_out / 16; p.unit_rows = 16; p.n_boxes = 1; p.k_chunks = n_in / kBK;
    p.n_groups = choose_groups(n_mb, p.units_total, G); p.n_rb = n_mb; p.rows = n; p.a_row_base = 0; p.a_part_rows = n;
    p.M = n; p.d = n_in; p.sumsq = sumsq; p.n_ss = n_ss; p.eps = c->cfg.rms_eps;
    p.lin_out = out; p.lin_n_out = n_out; p.lin_accumulate = accumulate ? 1 : 0;
    p.gamma_next = (const __nv_bfloat16 *)gamma_next; p.xg_next = xg_next; p.sumsq_out = sumsq_out;
    p.status = (int32_t *)(c->ws + c->lay.status); p.user_status = user_status;
    finish_shape(p, G / p.n_groups);
    if (n_ss_out) *n_ss_out = p.n_vr;
    if (!make_map(s, &mA, a, n_in, 2 * (uint64_t)n, 128) || !make_map(s, &mB, w, n_in, n_out, p.bn))
        return note_err(c, cudaErrorInvalidValue, "tensor map (module product)");
    c->launches++;
    return note_err(c, launch_tc<KIND_LIN, false>(mA, mB, mB, p, p.n_groups * p.n_vr, st, !(c->cfg.flags & MRP_FLAG_NO_PDL)),
                    "module product kernel");
}

// Three products over the same operand rows in one launch: out_i[n, n_out] = rstd(row) * (A W_i^T), i = 0, 1, 2
// (q, k, v of a module layer).  The weight-row ranges are dealt out per matrix, so a CTA's tile is three times as
// wide as with a launch per matrix, and the activation tiles are loaded a third as often per weight byte.
cudaError_t tc_linear3(Ctx *c, const __nv_bfloat16 *a, int n, int n_in, const void *w0, const void *w1, const void *w2,
                       int n_out, const float *sumsq, int n_ss, float *out0, float *out1, float *out2, int32_t *user_status,
                       cudaStream_t st)
{
    const TcState *s = (const TcState *)c->tc_state;
    const int G = c->sm_count, n_mb = (n + 127) / 128;
    CUtensorMap mA, mB0, mB1, mB2;
    TcParams p;
    memset(&p, 0, sizeof(p));
    p.units_total = n_out / 16; p.unit_rows = 16; p.n_boxes = 1; p.k_chunks = n_in / kBK;
    p.n_groups = choose_groups(n_mb, 3 * p.units_total, G); p.n_rb = n_mb; p.rows = n; p.a_row_base = 0; p.a_part_rows = n;
    p.M = n; p.d = n_in; p.sumsq = sumsq; p.n_ss = n_ss; p.eps = c->cfg.rms_eps;
    p.lin_out = out0; p.lin_out1 = out1; p.lin_out2 = out2; p.lin_n_out = n_out; p.lin_nw = 3;
    p.status = (int32_t *)(c->ws + c->lay.status); p.user_status = user_status;
    int per_w = (G / p.n_groups) / 3;                    // weight-row ranges per matrix
    if (per_w < 1) per_w = 1;
    finish_shape(p, per_w);
    p.n_vr = 3 * per_w;
    if (!make_map(s, &mA, a, n_in, 2 * (uint64_t)n, 128) || !make_map(s, &mB0, w0, n_in, n_out, p.bn) ||
        !make_map(s, &mB1, w1, n_in, n_out, p.bn) || !make_map(s, &mB2, w2, n_in, n_out, p.bn))
        return note_err(c, cudaErrorInvalidValue, "tensor map (module q, k, v)");
    c->launches++;
    return note_err(c, launch_tc<KIND_LIN, false>(mA, mB0, mB1, p, p.n_groups * p.n_vr, st, !(c->cfg.flags & MRP_FLAG_NO_PDL), &mB2),
                    "module q, k, v kernel");
}

// act[n, F] (bf16 hi rows, lo rows n * F elements further on) = silu(rstd * A Wg^T) * (rstd * A Wu^T): the head
// chain's gate/up kernel on other operands.
cudaError_t tc_gate_up(Ctx *c, const __nv_bfloat16 *a, int n, int n_in, const void *w_gate, const void *w_up, int F,
                       const float *sumsq, int n_ss, __nv_bfloat16 *act, int32_t *user_status, cudaStream_t st)
{
    const TcState *s = (const TcState *)c->tc_state;
    const int G = c->sm_count, n_mb = (n + 127) / 128;
    CUtensorMap mA, mB0, mB1;
    TcParams p;
    memset(&p, 0, sizeof(p));
    p.units_total = F / 8; p.unit_rows = 8; p.n_boxes = 2; p.k_chunks = n_in / kBK;
    p.n_groups = choose_groups(n_mb, p.units_total, G); p.n_rb = n_mb; p.rows = n; p.a_row_base = 0; p.a_part_rows = n;
    p.M = n; p.d = n_in; p.F = F;
    p.sumsq = sumsq; p.n_ss = n_ss; p.eps = c->cfg.rms_eps; p.act = act;
    p.status = (int32_t *)(c->ws + c->lay.status); p.user_status = user_status;
    finish_shape(p, G / p.n_groups);
    if (!make_map(s, &mA, a, n_in, 2 * (uint64_t)n, 128) || !make_map(s, &mB0, w_gate, n_in, F, p.bn / 2) ||
        !make_map(s, &mB1, w_up, n_in, F, p.bn / 2))
        return note_err(c, cudaErrorInvalidValue, "tensor map (module gate/up)");
    c->launches++;
    return note_err(c, launch_tc<KIND_GU, false>(mA, mB0, mB1, p, p.n_groups * p.n_vr, st, !(c->cfg.flags & MRP_FLAG_NO_PDL)),
                    "module gate/up kernel");
}

cudaError_t tc_draft(Ctx *c, const void *hidden, const float *logits0, const int32_t *row_index, int M,
                     int K, const mrp_draft_out &out, cudaStream_t st)
{
    if (M == 0) return cudaSuccess;
    if (K == 0) return simt_draft(c, hidden, logits0, row_index, M, K, out, st);
    const TcState *s = (const TcState *)c->tc_state;
    const int d = c->cfg.d, F = c->cfg.d_ff, V = c->cfg.vocab;
    const int G = c->sm_count;
    float *h0f = (float *)(c->ws + c->lay.h0f), *hcur = (float *)(c->ws + c->lay.hcur);
    __nv_bfloat16 *xg = (__nv_bfloat16 *)(c->ws + c->lay.xg), *act = (__nv_bfloat16 *)(c->ws + c->lay.act);
    __nv_bfloat16 *xt = (__nv_bfloat16 *)(c->ws + c->lay.xt);
    float *sumsq = (float *)(c->ws + c->lay.sumsq);
    Partial *partials = (Partial *)(c->ws + c->lay.partials);
    int32_t *status = (int32_t *)(c->ws + c->lay.status);
    if (G > kSumsqSlices || G > c->lay.n_slices_max)
        return note_err(c, cudaErrorInvalidValue, "workspace slices");
    const int n_mb = (M + 127) / 128;
    // The head GEMMs can run on CTA pairs like the LM head (see tc_lm_tail), but gain nothing from it: with
    // two MMA passes per loaded tile (bf16 hi + lo) they are bound by the tensor pipe, not by the tile feed.
    const bool pair = false;
    const int n_cta = pair ? G / 2 : G, n_blk = pair ? (n_mb + 1) / 2 : n_mb;

    const TcPlan pl = tc_plan(c, M, K, out, st, true);
    const int n_rs = pl.n_rs;
    const bool pdl = pl.pdl, few_rows = pl.few_rows, f16_lm = pl.f16_lm, chain = pl.chain;

    prof_mark(c, 0, st);
    cudaError_t e = note_err(c, launch_k(tc_prep_kernel, dim3(M), dim3(256), 0, st, !(c->cfg.flags & MRP_FLAG_NO_PDL),
                                         (const __nv_bfloat16 *)hidden, row_index, d, c->lo_x, c->lo_xt,
                                      (const __nv_bfloat16 *)c->heads[0].rms_gamma, h0f, hcur, xg, xt, sumsq,
                                      (int32_t *)(c->ws + c->lay.sk_counters), kSkMaxTiles,
                                      (unsigned long long *)(c->ws + c->lay.ssq_fix), c->from_hidden ? 1 : 0,
                                      (const __nv_bfloat16 *)c->final_gamma, c->cfg.rms_eps,
                                      (c->from_hidden && f16_lm) ? (__half *)(c->ws + c->lay.xt16) : (__half *)nullptr,
                                      c->input_rows, status, out.status),
                             "tc_prep_kernel");
    c->launches++;
    if (e != cudaSuccess) return e;

    int n_ss = 1;
    bool chain_done = false;
    if (chain) {
        e = sk_chain(c, M, K, out, st, f16_lm, false);
        if (e != cudaSuccess) return e;
        chain_done = true;
    }
    for (int k = 1; k <= K && !chain_done; ++k) {
        if (few_rows) {
            e = sk_gateup(c, k, M, K, n_ss, out, st, pdl);
            if (e != cudaSuccess) return e;
            e = sk_down(c, k, M, K, out, st, pdl, &n_ss, f16_lm);
            if (e != cudaSuccess) return e;
            continue;
        }
        const mrp_head_weights &hw = c->heads[k - 1];
        CUtensorMap mA, mB0, mB1;
        // gate/up + SwiGLU
        TcParams p;
        memset(&p, 0, sizeof(p));
        p.units_total = F / 8; p.unit_rows = 8; p.n_boxes = 2; p.k_chunks = d / kBK;
        p.n_groups = choose_groups(n_blk, p.units_total, n_cta); p.n_rb = n_blk; p.rows = M; p.a_row_base = 0; p.a_part_rows = M;
        p.M = M; p.K = K; p.V = V; p.d = d; p.F = F; p.n_rs = n_rs;
        p.sumsq = sumsq; p.n_ss = n_ss; p.eps = c->cfg.rms_eps; p.act = act;
        p.status = status; p.user_status = out.status;
        finish_shape(p, n_cta / p.n_groups, 2, pair);
        if (!make_map(s, &mA, xg, d, 2 * (uint64_t)M, 128) || !make_map(s, &mB0, hw.w_gate, d, F, p.bn / 2) ||
            !make_map(s, &mB1, hw.w_up, d, F, p.bn / 2))
            return note_err(c, cudaErrorInvalidValue, "tensor map (gate/up)");
        e = note_err(c, pair ? launch_tc<KIND_GU, false, false, false, true>(mA, mB0, mB1, p, 2 * p.n_groups * p.n_vr, st, pdl)
                             : launch_tc<KIND_GU, false>(mA, mB0, mB1, p, p.n_groups * p.n_vr, st, pdl), "gate/up kernel");
        c->launches++;
        if (e != cudaSuccess) return e;
        // down projection, residual add, next operands
        memset(&p, 0, sizeof(p));
        p.units_total = d / 16; p.unit_rows = 16; p.n_boxes = 1; p.k_chunks = F / kBK;
        p.n_groups = choose_groups(n_blk, p.units_total, n_cta); p.n_rb = n_blk; p.rows = M;
        p.M = M; p.K = K; p.V = V; p.d = d; p.F = F; p.n_rs = n_rs; p.a_part_rows = M;
        p.hcur = hcur; p.h0f = h0f;
        p.gamma_next = (k < K) ? (const __nv_bfloat16 *)c->heads[k].rms_gamma : nullptr;
        p.xg_next = (k < K) ? xg : nullptr;
        p.xt_k = xt + (size_t)k * M * d;
        p.xt16_k = f16_lm ? (__half *)(c->ws + c->lay.xt16) + (size_t)(k - (c->from_hidden ? 0 : 1)) * M * d : nullptr;
        p.sumsq_out = sumsq;
        p.hidden_out = (k == K) ? out.hidden_out : nullptr;
        p.status = status; p.user_status = out.status;
        finish_shape(p, n_cta / p.n_groups, 2, pair);
        if (!make_map(s, &mA, act, F, 2 * (uint64_t)M, 128) || !make_map(s, &mB0, hw.w_down, F, d, pair ? p.bn / 2 : p.bn))
            return note_err(c, cudaErrorInvalidValue, "tensor map (down)");
        e = note_err(c, pair ? launch_tc<KIND_DN, false, false, false, true>(mA, mB0, mB0, p, 2 * p.n_groups * p.n_vr, st, pdl)
                             : launch_tc<KIND_DN, false>(mA, mB0, mB0, p, p.n_groups * p.n_vr, st, pdl), "down kernel");
        c->launches++;
        if (e != cudaSuccess) return e;
        n_ss = p.n_vr;
    }
    return tc_lm_tail(c, pl, logits0, row_index, M, K, out, st);
}

}  // namespace mrp
