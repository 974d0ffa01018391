// Tensor-core kernel family (sm_100a): tcgen05.mma with TMEM accumulators, operands staged in
// shared memory by TMA (128-byte swizzle), warp-specialised: one TMA producer thread, one MMA
// issuer thread, four epilogue warps that read the accumulators back with tcgen05.ld.
//
// All three GEMMs of the drafting pass share one main loop and differ in the epilogue:
//   GU  gate/up projections of a head:  act = silu(rstd * Wg x) * (rstd * Wu x)          (a1)
//   DN  down projection:  h <- h + Wd act, emits the bf16 operands of the next GEMMs      (a1)
//   LM  shared LM head on the stacked residual rows h_k - h_0, fused with "+ l_0" and the
//       online softmax statistics (max, sum of exponentials, argmax, runner-up)      (a2, a3)
// Precision: weights are exact bf16; every activation operand (head input, SwiGLU output, stacked
// residual rows) is carried as a pair of bf16 matrices hi + lo (lo = bf16 of what hi lost), and
// each weight tile is multiplied by both, so the products are exact to about 2^-17 and the
// fp32 accumulators stay within the 2e-3 tolerance on confidence / log-sum-exp.
// Orientation: activation rows are the MMA M dimension (128 TMEM lanes, one row per epilogue
// thread), weight rows are the MMA N dimension.  Every CTA owns a contiguous range of weight
// rows, split into equal tiles, and streams it exactly once per 128-row activation block.
#include <cuda.h>
#include <limits.h>
#include <string.h>

#include <new>

#include "mrp_internal.cuh"

namespace mrp {
namespace {

constexpr int kThreads = 192;
constexpr int kBK = 64;                    // bf16 elements per k-chunk = one 128-byte swizzle row
constexpr int kATile = 128 * 128;          // bytes of a 128-row A tile
constexpr int kAccCols = 256;              // TMEM columns per accumulator buffer (two buffers)
constexpr int kSmemBudget = 230000;        // dynamic shared memory we ask for at most
constexpr long long kWaitCycles = 3000000000LL;   // bound on any barrier wait (about 1.5 s)

enum { KIND_GU = 0, KIND_DN = 1, KIND_LM = 2 };

struct TcParams {
    // decomposition of the weight rows (MMA N)
    int units_total;     // weight-row extent in units
    int unit_rows;       // rows per unit per B box (LM/DN 16, GU 8 of gate + 8 of up)
    int w_units;         // tile width in units
    int bn;              // MMA N = rows of the B tile
    int n_boxes;         // TMA boxes per B tile (GU 2, else 1)
    int k_chunks;        // contraction extent / 64
    int n_stages;
    int n_mb;            // 128-row activation blocks
    int a_row_base;      // A row coordinate of accumulator 0, block 0 (hi part)
    int a_row_step;      // A row offset between accumulators
    int a_part_rows;     // A row offset from the hi part to the lo part
    int M, K, V, d, F;
    int stacked;         // LM: all (K+1)*M row-steps in one block
    int n_rs;            // LM: (K+1)*M
    // LM
    const float *logits0;
    const int32_t *row_index;
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
    float *sumsq_out;
    float *hidden_out;
    int32_t *status;
    int32_t *user_status;
};

// ---------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: gives up after kWaitCycles or when another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                          const TcParams &p)
{
    if (mbar_try_wait(bar, parity)) return true;
    long long t0 = clock64();
    uint32_t spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 255u) == 0) {
            if (*abort_flag) return false;
            if (clock64() - t0 > kWaitCycles) {
                *abort_flag = 1;
                atomicOr(p.status, MRP_DEV_TIMEOUT);
                if (p.user_status) atomicOr(p.user_status, MRP_DEV_TIMEOUT);
                return false;
            }
        }
    }
    return true;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int c0, int c1, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap *map)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t da, uint64_t db, uint32_t idesc, uint32_t acc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(da), "l"(db), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float *v)
{
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float *v)
{
    uint32_t r[8];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ float ex2f(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float4 ldg_nc4(const float *p)
{
    float4 v;
    asm volatile("ld.global.nc.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
    return v;
}

// Shared-memory matrix descriptor of a K-major bf16 tile whose rows are 128 bytes, stored with
// the 128-byte swizzle in 8-row groups of 1024 bytes (what a SWIZZLE_128B TMA box writes).
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr)
{
    uint64_t desc = 0;
    desc |= (uint64_t)((saddr & 0x3FFFFu) >> 4);        // start address, 16-byte units
    desc |= (uint64_t)1 << 16;                          // leading byte offset (unused with swizzle)
    desc |= (uint64_t)(1024 >> 4) << 32;                // stride byte offset: 8-row group pitch
    desc |= (uint64_t)1 << 46;                          // descriptor version (Blackwell)
    desc |= (uint64_t)2 << 61;                          // layout type: 128-byte swizzle
    return desc;
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = bn.
__device__ __forceinline__ uint32_t make_idesc(int bn)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}

constexpr float kLog2e = 1.4426950408889634f;

// Online softmax statistics of one logit row, updated 16 columns at a time.
struct RowStat {
    float mx, sum, second;
    int idx;
    __device__ __forceinline__ void init() { mx = -INFINITY; sum = 0.f; second = -INFINITY; idx = INT_MAX; }
    template <bool MARGIN>
    __device__ __forceinline__ void update(const float *l, int v_base)
    {
        float cmax = l[0];
#pragma unroll
        for (int j = 1; j < 16; ++j) cmax = fmaxf(cmax, l[j]);
        if (cmax > mx) {
            int jj = 15;
#pragma unroll
            for (int j = 14; j >= 0; --j) jj = (l[j] == cmax) ? j : jj;
            if (MARGIN) {
                float c2 = -INFINITY;
#pragma unroll
                for (int j = 0; j < 16; ++j) c2 = (j != jj) ? fmaxf(c2, l[j]) : c2;
                second = fmaxf(mx, c2);
            }
            sum *= ex2f((mx - cmax) * kLog2e);
            mx = cmax;
            idx = v_base + jj;
        } else if (MARGIN) {
            second = fmaxf(second, cmax);
        }
        const float ms = mx * kLog2e;
        float s = 0.f;
#pragma unroll
        for (int j = 0; j < 16; ++j) s += ex2f(fmaf(l[j], kLog2e, -ms));
        sum += s;
    }
    __device__ __forceinline__ Partial partial() const
    {
        Partial p;
        p.mx = mx; p.sum = sum; p.idx = idx; p.second = second;
        return p;
    }
};

__device__ __forceinline__ void load16(const float *p, float *v)
{
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float4 x = ldg_nc4(p + 4 * i);
        v[4 * i] = x.x; v[4 * i + 1] = x.y; v[4 * i + 2] = x.z; v[4 * i + 3] = x.w;
    }
}
__device__ __forceinline__ void load16_rw(const float *p, float *v)   // data this kernel also writes
{
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float4 x = *reinterpret_cast<const float4 *>(p + 4 * i);
        v[4 * i] = x.x; v[4 * i + 1] = x.y; v[4 * i + 2] = x.z; v[4 * i + 3] = x.w;
    }
}
__device__ __forceinline__ void store16(float *p, const float *v)
{
#pragma unroll
    for (int i = 0; i < 4; ++i)
        *reinterpret_cast<float4 *>(p + 4 * i) = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
}
__device__ __forceinline__ uint32_t pack_bf16(float a, float b)
{
    __nv_bfloat162 t = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t *>(&t);
}
// hi = bf16(a, b); lo = bf16 of the rounding remainders.
__device__ __forceinline__ void split_bf16(float a, float b, uint32_t &hi, uint32_t &lo)
{
    const __nv_bfloat16 ha = __float2bfloat16_rn(a), hb = __float2bfloat16_rn(b);
    __nv_bfloat162 h;
    h.x = ha; h.y = hb;
    hi = *reinterpret_cast<uint32_t *>(&h);
    lo = pack_bf16(a - __bfloat162float(ha), b - __bfloat162float(hb));
}
// Stores n (8 or 16) values as bf16 hi at dst and bf16 lo at dst + lo_off.
template <int N>
__device__ __forceinline__ void store_split(__nv_bfloat16 *dst, size_t lo_off, const float *v)
{
    uint32_t hi[N / 2], lo[N / 2];
#pragma unroll
    for (int j = 0; j < N; j += 2) split_bf16(v[j], v[j + 1], hi[j >> 1], lo[j >> 1]);
    uint4 *dh = reinterpret_cast<uint4 *>(dst), *dl = reinterpret_cast<uint4 *>(dst + lo_off);
#pragma unroll
    for (int i = 0; i < N / 8; ++i) {
        dh[i] = make_uint4(hi[4 * i], hi[4 * i + 1], hi[4 * i + 2], hi[4 * i + 3]);
        dl[i] = make_uint4(lo[4 * i], lo[4 * i + 1], lo[4 * i + 2], lo[4 * i + 3]);
    }
}

// ---------------------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------------------
template <int KIND, int NACC, bool MARGIN>
__global__ void __launch_bounds__(kThreads, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB0,
               const __grid_constant__ CUtensorMap tmB1, const TcParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    // With one accumulator a stage holds the hi and the lo A tile and one B tile; with several
    // accumulators a stage holds one A tile per accumulator and the k-loop alternates hi / lo
    // (the B chunk is then fetched twice in a row, the second time from L2).
    constexpr bool SIS = (NACC == 1);
    constexpr int NA = SIS ? 2 : NACC;
    const int n_it = SIS ? p.k_chunks : 2 * p.k_chunks;
    const int b_bytes = (p.bn * 128 + 1023) & ~1023;
    const int stage_bytes = NA * kATile + b_bytes;
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
    const int cta = blockIdx.x, G = gridDim.x;
    const int u0 = (int)((long long)cta * p.units_total / G);
    const int u1 = (int)((long long)(cta + 1) * p.units_total / G);
    const int n_t = (u1 - u0 + p.w_units - 1) / p.w_units;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.n_stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 4); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        prefetch_tmap(&tmA);
        prefetch_tmap(&tmB0);
        if (KIND == KIND_GU) prefetch_tmap(&tmB1);
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_holder)), "r"(2u * kAccCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            const uint32_t tx = (uint32_t)(NA * kATile + p.bn * 128);
            const int box_rows = p.bn / p.n_boxes;
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            for (int mb = 0; mb < p.n_mb && ok; ++mb) {
                for (int t = 0; t < n_t && ok; ++t) {
                    const int n0 = (u0 + t * p.w_units) * p.unit_rows;
                    for (int it = 0; it < n_it; ++it) {
                        const int kk = SIS ? it : (it >> 1);
                        if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, p)) { ok = false; break; }
                        mbar_expect_tx(full_bar(s), tx);
                        const uint32_t sa = base + (uint32_t)s * stage_bytes;
                        if (SIS) {
                            tma_load_2d(sa, &tmA, kk * kBK, p.a_row_base + mb * 128, full_bar(s));
                            tma_load_2d(sa + kATile, &tmA, kk * kBK, p.a_part_rows + p.a_row_base + mb * 128,
                                        full_bar(s));
                        } else {
                            const int part_row = (it & 1) * p.a_part_rows;
#pragma unroll
                            for (int a = 0; a < NACC; ++a)
                                tma_load_2d(sa + a * kATile, &tmA, kk * kBK,
                                            part_row + p.a_row_base + a * p.a_row_step + mb * 128, full_bar(s));
                        }
                        const uint32_t sb = sa + NA * kATile;
                        tma_load_2d(sb, &tmB0, kk * kBK, n0, full_bar(s));
                        if (KIND == KIND_GU)
                            tma_load_2d(sb + box_rows * 128, &tmB1, kk * kBK, n0, full_bar(s));
                        if (++s == p.n_stages) { s = 0; ph ^= 1u; }
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            const uint32_t idesc = make_idesc(p.bn);
            int s = 0, acc = 0;
            uint32_t ph = 0, acc_ph = 0;
            bool ok = true;
            for (int mb = 0; mb < p.n_mb && ok; ++mb) {
                for (int t = 0; t < n_t && ok; ++t) {
                    if (!mbar_wait(tempty_bar(acc), acc_ph ^ 1u, abort_flag, p)) { ok = false; break; }
                    tc_fence_after();
                    for (int it = 0; it < n_it; ++it) {
                        if (!mbar_wait(full_bar(s), ph, abort_flag, p)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t sa = base + (uint32_t)s * stage_bytes;
                        const uint64_t db = make_smem_desc(sa + NA * kATile);
#pragma unroll
                        for (int a = 0; a < NA; ++a) {
                            const uint64_t da = make_smem_desc(sa + a * kATile);
                            const uint32_t dt = tmem_base + (uint32_t)(acc * kAccCols + (SIS ? 0 : a * p.bn));
#pragma unroll
                            for (int k4 = 0; k4 < kBK / 16; ++k4)
                                umma_bf16(dt, da + 2u * k4, db + 2u * k4, idesc,
                                          (it > 0 || k4 > 0 || (SIS && a > 0)) ? 1u : 0u);
                        }
                        umma_commit(empty_bar(s));
                        if (++s == p.n_stages) { s = 0; ph ^= 1u; }
                    }
                    if (!ok) break;
                    umma_commit(tfull_bar(acc));
                    acc ^= 1;
                    if (acc == 0) acc_ph ^= 1u;
                }
            }
        }
    } else {
        // ---------------- epilogue warps (TMEM lane quadrant = warp % 4) ----------------
        const int q = warp & 3;
        const int r = q * 32 + lane;
        const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
        int acc = 0;
        uint32_t acc_ph = 0;
        bool ok = true;
        for (int mb = 0; mb < p.n_mb && ok; ++mb) {
            // ---- per-block state ----
            const int m_or_rs = mb * 128 + r;
            RowStat st[KIND == KIND_LM ? NACC + 1 : 1];
            bool valid = false;
            const float *l0p = nullptr;
            int k_of_row = 0, m_of_row = 0;
            float rstd = 0.f, ssq = 0.f;
            if (KIND == KIND_LM) {
#pragma unroll
                for (int i = 0; i < NACC + 1; ++i) st[i].init();
                if (p.stacked) {
                    valid = m_or_rs < p.n_rs;
                    if (valid) { k_of_row = m_or_rs / p.M; m_of_row = m_or_rs - k_of_row * p.M; }
                } else {
                    valid = m_or_rs < p.M;
                    m_of_row = m_or_rs;
                }
                if (valid) {
                    const size_t row = p.row_index ? (size_t)p.row_index[m_of_row] : (size_t)m_of_row;
                    l0p = p.logits0 + row * (size_t)p.V;
                }
            } else {
                valid = m_or_rs < p.M;
                m_of_row = m_or_rs;
                if (KIND == KIND_GU && valid) {
                    float s = 0.f;
                    for (int i = 0; i < p.n_ss; ++i) s += p.sumsq[(size_t)i * p.M + m_of_row];
                    rstd = rsqrtf(s / (float)p.d + p.eps);
                }
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
                        float l0[16], a[16], l[16];
                        if (valid) load16(l0p + v, l0);
                        if (p.stacked) {
                            tmem_ld16(tacc + c * 16, a);
                            if (valid) {
#pragma unroll
                                for (int j = 0; j < 16; ++j) l[j] = (k_of_row > 0) ? l0[j] + a[j] : l0[j];
                                st[0].template update<MARGIN>(l, v);
                                if (p.logits_out && k_of_row > 0)
                                    store16(p.logits_out + ((size_t)(m_or_rs - p.M)) * p.V + v, l);
                            }
                        } else {
                            if (valid) st[0].template update<MARGIN>(l0, v);
#pragma unroll
                            for (int s = 0; s < NACC; ++s) {
                                tmem_ld16(tacc + s * p.bn + c * 16, a);
                                if (valid) {
#pragma unroll
                                    for (int j = 0; j < 16; ++j) l[j] = l0[j] + a[j];
                                    st[s + 1].template update<MARGIN>(l, v);
                                    if (p.logits_out)
                                        store16(p.logits_out + ((size_t)s * p.M + m_of_row) * p.V + v, l);
                                }
                            }
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
                if (lane == 0) mbar_arrive(tempty_bar(acc));
                acc ^= 1;
                if (acc == 0) acc_ph ^= 1u;
            }
            // ---- per-block results ----
            if (ok && valid) {
                if (KIND == KIND_LM) {
                    if (p.stacked) {
                        p.partials[(size_t)cta * p.n_rs + m_or_rs] = st[0].partial();
                    } else {
#pragma unroll
                        for (int s = 0; s < NACC + 1; ++s)
                            p.partials[(size_t)cta * p.n_rs + (size_t)s * p.M + m_of_row] = st[s].partial();
                    }
                } else if (KIND == KIND_DN) {
                    p.sumsq_out[(size_t)cta * p.M + m_of_row] = ssq;
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
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(2u * kAccCols) : "memory");
    }
}

// Gather masked rows: fp32 copies of h_0, the first head's operand bf16(h_0 * gamma_1), the
// row sums of squares, and the zero rows that stand for step 0 in the stacked LM-head operand.
__global__ void tc_prep_kernel(const __nv_bfloat16 *__restrict__ hidden, const int32_t *__restrict__ row_index,
                               int d, int M, int n_rs, const __nv_bfloat16 *__restrict__ gamma1,
                               float *__restrict__ h0f, float *__restrict__ hcur, __nv_bfloat16 *__restrict__ xg,
                               __nv_bfloat16 *__restrict__ xt0, float *__restrict__ sumsq)
{
    __shared__ float red[8];
    const int m = blockIdx.x;
    const size_t row = row_index ? (size_t)row_index[m] : (size_t)m;
    float ss = 0.f;
    for (int j = threadIdx.x; j < d; j += blockDim.x) {
        const float v = __bfloat162float(hidden[row * d + j]);
        const size_t o = (size_t)m * d + j;
        h0f[o] = v;
        hcur[o] = v;
        if (gamma1) {
            const float x = v * __bfloat162float(gamma1[j]);
            const __nv_bfloat16 hi = __float2bfloat16_rn(x);
            xg[o] = hi;
            xg[(size_t)M * d + o] = __float2bfloat16_rn(x - __bfloat162float(hi));
        }
        xt0[o] = __float2bfloat16(0.f);
        xt0[(size_t)n_rs * d + o] = __float2bfloat16(0.f);
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
    }
}

// ---------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

struct TcState {
    EncodeTiledFn encode;
};

// bf16 row-major [rows, inner] matrix, box = [box_rows, 64 elements], 128-byte swizzle,
// out-of-range elements read as zero.
bool make_map(const TcState *s, CUtensorMap *map, const void *ptr, uint64_t inner, uint64_t rows, uint32_t box_rows)
{
    cuuint64_t dims[2] = {inner, rows};
    cuuint64_t strides[1] = {inner * 2};
    cuuint32_t box[2] = {(cuuint32_t)kBK, box_rows};
    cuuint32_t es[2] = {1, 1};
    return s->encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims, strides, box, es,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tile width (in units, at most w_max) for CTAs owning up to `maxunits` units: the width that
// wastes the fewest rows beyond the range, the wider one on ties.
int choose_tile_units(int maxunits, int w_max)
{
    int best_w = 1, best_waste = INT_MAX;
    for (int w = 1; w <= w_max; ++w) {
        const int T = (maxunits + w - 1) / w;
        const int waste = T * w - maxunits;
        if (waste <= best_waste) { best_waste = waste; best_w = w; }
    }
    return best_w;
}

void finish_shape(TcParams &p, int nacc, int grid)
{
    const int maxunits = (p.units_total + grid - 1) / grid;
    const int bn_max = kAccCols / nacc;
    const int rows_per_unit = p.unit_rows * p.n_boxes;
    int w_max = bn_max / rows_per_unit;
    if (w_max > 256 / rows_per_unit) w_max = 256 / rows_per_unit;
    if (w_max < 1) w_max = 1;
    p.w_units = choose_tile_units(maxunits < 1 ? 1 : maxunits, w_max);
    p.bn = p.w_units * rows_per_unit;
    const int b_bytes = (p.bn * 128 + 1023) & ~1023;
    const int stage = (nacc == 1 ? 2 : nacc) * kATile + b_bytes;
    int ns = (kSmemBudget - 1024 - 512) / stage;
    if (ns > 12) ns = 12;
    p.n_stages = ns;
}

size_t smem_bytes(const TcParams &p, int nacc)
{
    const int b_bytes = (p.bn * 128 + 1023) & ~1023;
    return (size_t)p.n_stages * ((nacc == 1 ? 2 : nacc) * kATile + b_bytes) + 1024 + 8 * (2 * p.n_stages + 4) + 16;
}

template <int KIND, int NACC, bool MARGIN>
cudaError_t launch_tc(const CUtensorMap &a, const CUtensorMap &b0, const CUtensorMap &b1, const TcParams &p,
                      int grid, cudaStream_t st)
{
    auto kern = tc_gemm_kernel<KIND, NACC, MARGIN>;
    const size_t smem = smem_bytes(p, NACC);
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    kern<<<grid, kThreads, smem, st>>>(a, b0, b1, p);
    return cudaGetLastError();
}

template <bool MARGIN>
cudaError_t launch_lm(int nacc, const CUtensorMap &a, const CUtensorMap &b, const TcParams &p, int grid, cudaStream_t st)
{
    switch (nacc) {
    case 1: return launch_tc<KIND_LM, 1, MARGIN>(a, b, b, p, grid, st);
    case 2: return launch_tc<KIND_LM, 2, MARGIN>(a, b, b, p, grid, st);
    case 3: return launch_tc<KIND_LM, 3, MARGIN>(a, b, b, p, grid, st);
    case 4: return launch_tc<KIND_LM, 4, MARGIN>(a, b, b, p, grid, st);
    default: return cudaErrorInvalidValue;
    }
}

}  // namespace

bool tc_supported(const mrp_config &cfg, const mrp_head_weights *heads, const void *w_lm)
{
    if (cfg.dtype != MRP_BF16) return false;
    if (cfg.d % 64 || cfg.d_ff % 64 || cfg.vocab % 16) return false;
    if (cfg.n_heads > 4) return false;
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
    return cudaSuccess;
}

void tc_destroy(Ctx *c)
{
    delete (TcState *)c->tc_state;
    c->tc_state = nullptr;
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

    prof_mark(c, 0, st);
    const int n_rs = (K + 1) * M;
    tc_prep_kernel<<<M, 256, 0, st>>>((const __nv_bfloat16 *)hidden, row_index, d, M, n_rs,
                                      (const __nv_bfloat16 *)c->heads[0].rms_gamma, h0f, hcur, xg, xt, sumsq);
    c->launches++;
    cudaError_t e = note_err(c, cudaGetLastError(), "tc_prep_kernel");
    if (e != cudaSuccess) return e;

    int n_ss = 1;
    for (int k = 1; k <= K; ++k) {
        const mrp_head_weights &hw = c->heads[k - 1];
        CUtensorMap mA, mB0, mB1;
        // gate/up + SwiGLU
        TcParams p;
        memset(&p, 0, sizeof(p));
        p.units_total = F / 8; p.unit_rows = 8; p.n_boxes = 2; p.k_chunks = d / kBK; p.n_mb = n_mb;
        p.a_row_base = 0; p.a_row_step = 0; p.a_part_rows = M;
        p.M = M; p.K = K; p.V = V; p.d = d; p.F = F; p.n_rs = n_rs;
        p.sumsq = sumsq; p.n_ss = n_ss; p.eps = c->cfg.rms_eps; p.act = act;
        p.status = status; p.user_status = out.status;
        finish_shape(p, 1, G);
        if (!make_map(s, &mA, xg, d, 2 * (uint64_t)M, 128) || !make_map(s, &mB0, hw.w_gate, d, F, p.bn / 2) ||
            !make_map(s, &mB1, hw.w_up, d, F, p.bn / 2))
            return note_err(c, cudaErrorInvalidValue, "tensor map (gate/up)");
        e = note_err(c, launch_tc<KIND_GU, 1, false>(mA, mB0, mB1, p, G, st), "gate/up kernel");
        c->launches++;
        if (e != cudaSuccess) return e;
        // down projection, residual add, next operands
        memset(&p, 0, sizeof(p));
        p.units_total = d / 16; p.unit_rows = 16; p.n_boxes = 1; p.k_chunks = F / kBK; p.n_mb = n_mb;
        p.M = M; p.K = K; p.V = V; p.d = d; p.F = F; p.n_rs = n_rs; p.a_part_rows = M;
        p.hcur = hcur; p.h0f = h0f;
        p.gamma_next = (k < K) ? (const __nv_bfloat16 *)c->heads[k].rms_gamma : nullptr;
        p.xg_next = (k < K) ? xg : nullptr;
        p.xt_k = xt + (size_t)k * M * d;
        p.sumsq_out = sumsq;
        p.hidden_out = (k == K) ? out.hidden_out : nullptr;
        p.status = status; p.user_status = out.status;
        finish_shape(p, 1, G);
        if (!make_map(s, &mA, act, F, 2 * (uint64_t)M, 128) || !make_map(s, &mB0, hw.w_down, F, d, p.bn))
            return note_err(c, cudaErrorInvalidValue, "tensor map (down)");
        e = note_err(c, launch_tc<KIND_DN, 1, false>(mA, mB0, mB0, p, G, st), "down kernel");
        c->launches++;
        if (e != cudaSuccess) return e;
        n_ss = G;
    }
    prof_mark(c, 1, st);
    {
        CUtensorMap mA, mB;
        TcParams p;
        memset(&p, 0, sizeof(p));
        const bool stacked = n_rs <= 128;
        const int nacc = stacked ? 1 : K;
        p.units_total = V / 16; p.unit_rows = 16; p.n_boxes = 1; p.k_chunks = d / kBK;
        p.n_mb = stacked ? 1 : n_mb;
        p.a_row_base = stacked ? 0 : M; p.a_row_step = stacked ? 0 : M; p.a_part_rows = n_rs;
        p.M = M; p.K = K; p.V = V; p.d = d; p.F = F; p.stacked = stacked ? 1 : 0; p.n_rs = n_rs;
        p.logits0 = logits0; p.row_index = row_index; p.partials = partials; p.logits_out = out.logits_out;
        p.status = status; p.user_status = out.status;
        finish_shape(p, nacc, G);
        if (!make_map(s, &mA, xt, d, 2 * (uint64_t)n_rs, 128) || !make_map(s, &mB, c->w_lm, d, V, p.bn))
            return note_err(c, cudaErrorInvalidValue, "tensor map (LM head)");
        e = note_err(c, out.margin ? launch_lm<true>(nacc, mA, mB, p, G, st)
                                   : launch_lm<false>(nacc, mA, mB, p, G, st), "LM-head kernel");
        c->launches++;
        if (e != cudaSuccess) return e;
    }
    prof_mark(c, 2, st);
    e = launch_combine(c, partials, G, (K + 1) * M, out, status, st);
    prof_mark(c, 3, st);
    return e;
}

}  // namespace mrp
