// Pieces shared by the tensor-core kernel files: PTX wrappers (mbarrier, TMA, tcgen05), shared
// memory / instruction descriptors, bf16 hi+lo splitting, tensor-map encoding.
#pragma once
#include <cuda.h>
#include <limits.h>

#include "mrp_internal.cuh"

namespace mrp {
namespace {

constexpr int kBK = 64;                    // bf16 elements per k-chunk = one 128-byte swizzle row
constexpr int kSmemBudget = 230000;        // dynamic shared memory we ask for at most
constexpr long long kWaitCycles = 3000000000LL;   // bound on any barrier wait (about 1.5 s)

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
template <typename P>
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                          const P &p)
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
// Same with an L2 eviction-priority hint (policy from l2_policy_*): weights that are read once
// per pass should not push the small, hot buffers (and the kernels' code) out of L2.
__device__ __forceinline__ void tma_load_2d_hint(uint32_t dst, const CUtensorMap *map, int c0, int c1, uint32_t bar,
                                                 uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "l"(policy) : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_evict_first()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    return pol;
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
// The same MMA on 8-bit floating-point operands (kind::f8f6f4; here both operands e4m3, 32 elements of
// the contraction per instruction).
__device__ __forceinline__ void umma_f8(uint32_t d_tmem, uint64_t da, uint64_t db, uint32_t idesc, uint32_t acc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(da), "l"(db), "r"(idesc), "r"(acc) : "memory");
}
// ---- CTA pairs (a cluster of two CTAs working on one 256-row MMA tile, cta_group::2) ----------------
// Shared-memory addresses carry the CTA's rank within the cluster in bit 24; clearing it names the same
// offset in the pair's leader (rank 0).
constexpr uint32_t kLeaderMask = 0xFEFFFFFFu;
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// All threads of both CTAs meet (release / acquire at cluster scope).
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// TMA load into this CTA's shared memory whose completion is counted by the LEADER's barrier at `bar`'s offset
// (no multicast: every CTA fetches its own tiles).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, int c0, int c1, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar & kLeaderMask), "r"(c0), "r"(c1) : "memory");
}
// 256 x N x 16 MMA over the pair: rows 0-127 of A from the leader's shared memory, 128-255 from the peer's;
// each CTA holds N / 2 rows of B; each CTA's tensor memory receives its 128 rows of D.  Issued by the leader.
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t da, uint64_t db, uint32_t idesc, uint32_t acc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(da), "l"(db), "r"(idesc), "r"(acc) : "memory");
}
// Arrival on the barrier at `bar`'s offset in BOTH CTAs once the pair's MMAs issued so far have completed.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((unsigned short)3) : "memory");
}
// Arrival on the leader's barrier from either CTA of the pair.
__device__ __forceinline__ void mbar_arrive_leader(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar & kLeaderMask) : "memory");
}
// Instruction descriptor of the pair's MMA: M = 256, N = bn, fp32 accumulation; bf16 (1) or fp16 (0) operands.
__device__ __forceinline__ uint32_t make_idesc_pair(int bn, bool f16)
{
    return (1u << 4) | (f16 ? 0u : ((1u << 7) | (1u << 10))) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
}

// True in exactly one lane of a converged warp, the same lane every time.  The MMA issuer runs
// its loop with the whole warp and only issues from the elected lane: the loop's barrier waits,
// fences and commits cost about half as many cycles that way as in a one-lane branch
// (measured per 64-element k-chunk of a 128 x 32 MMA: about 250 against 560 cycles), and a
// 128 x 256 x 16 MMA issues at the tensor pipe's own rate of 128 cycles instead of 139.
__device__ __forceinline__ bool elect_one()
{
    uint32_t r;
    asm volatile("{\n\t.reg .pred q;\n\telect.sync _|q, 0xffffffff;\n\tselp.u32 %0, 1, 0, q;\n\t}" : "=r"(r));
    return r != 0;
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

// Same, fp16 x fp16 -> fp32.
__device__ __forceinline__ uint32_t make_idesc_f16(int bn)
{
    return (1u << 4) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}
// Same for kind::f8f6f4 with both operands e4m3 (operand format code 0) -> fp32.
__device__ __forceinline__ uint32_t make_idesc_e4m3(int bn)
{
    return (1u << 4) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}

// e4m3 (the 8-bit floating-point format with 4 exponent bits of bias 7 and 3 mantissa bits; no
// infinities, largest finite value 448 = 0x7E, 0x7F = NaN; exponent field 0 = subnormals of spacing
// 2^-9): round to nearest, ties to even, saturating.
__device__ __forceinline__ uint32_t f32_to_e4m3(float x)
{
    const uint32_t sign = (__float_as_uint(x) >> 24) & 0x80u;
    const float a = fabsf(x);
    if (!(a <= 448.f)) return sign | 0x7Eu;
    if (a < 0.015625f) return sign | (uint32_t)__float2int_rn(a * 512.f);     // 0..8; 8 is the smallest normal
    uint32_t ua = __float_as_uint(a);
    ua += 0x7FFFFu + ((ua >> 20) & 1u);          // round the 23-bit mantissa to 3 bits, ties to even
    return sign | ((((ua >> 23) - 120u) << 3) | ((ua >> 20) & 7u));
}
__device__ __forceinline__ float e4m3_to_f32(uint32_t b)
{
    const int e = (b >> 3) & 15, m = b & 7;
    const float v = e ? __uint_as_float(((uint32_t)(e + 120) << 23) | ((uint32_t)m << 20)) : (float)m * 0.001953125f;
    return (b & 0x80u) ? -v : v;
}
// Power of two s = 2^E, E the smallest integer with amax <= 448 * 2^E (1 for amax = 0): the scale that
// maps a row onto the e4m3 range.
__device__ __forceinline__ float e4m3_row_scale(float amax)
{
    if (!(amax > 0.f)) return 1.f;
    int e;
    const float f = frexpf(amax, &e);            // amax = f * 2^e, f in [0.5, 1); 448 = 0.875 * 2^9
    return ldexpf(1.f, e - 9 + (f > 0.875f ? 1 : 0));
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

// Online partial sums of the KL objective of one row (teacher logits t against corrected logits l),
// updated 16 columns at a time: mx = running max of t, sum = sum exp(t - mx), cross = sum exp(t - mx) (t - l).
struct KlStat {
    float mx, sum, cross;
    __device__ __forceinline__ void init() { mx = -INFINITY; sum = 0.f; cross = 0.f; }
    __device__ __forceinline__ void update(const float *t, const float *l)
    {
        float cmax = t[0];
#pragma unroll
        for (int j = 1; j < 16; ++j) cmax = fmaxf(cmax, t[j]);
        if (cmax > mx) {
            const float sc = ex2f((mx - cmax) * kLog2e);
            sum *= sc;
            cross *= sc;
            mx = cmax;
        }
        const float ms = mx * kLog2e;
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            const float e = ex2f(fmaf(t[j], kLog2e, -ms));
            sum += e;
            cross = fmaf(e, t[j] - l[j], cross);
        }
    }
    __device__ __forceinline__ KlPartial partial() const
    {
        KlPartial p;
        p.mx = mx; p.sum = sum; p.cross = cross; p.pad = 0.f;
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
// 16 consecutive bf16 values (32-byte aligned address) as floats
__device__ __forceinline__ void load16_bf16(const __nv_bfloat16 *p, float *v)
{
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        uint4 q;
        asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(q.x), "=r"(q.y), "=r"(q.z), "=r"(q.w) : "l"(p + 8 * i));
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            v[8 * i + 2 * j] = __uint_as_float(w[j] << 16);
            v[8 * i + 2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
        }
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

}  // namespace

// ---------------------------------------------------------------------------------------
// Tensor maps
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
inline bool make_map(const TcState *s, CUtensorMap *map, const void *ptr, uint64_t inner, uint64_t rows,
                     uint32_t box_rows)
{
    cuuint64_t dims[2] = {inner, rows};
    cuuint64_t strides[1] = {inner * 2};
    cuuint32_t box[2] = {(cuuint32_t)kBK, box_rows};
    cuuint32_t es[2] = {1, 1};
    return s->encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims, strides, box, es,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 8-bit row-major [rows, inner] matrix, box = [box_rows, 128 bytes], 128-byte swizzle.
inline bool make_map_u8(const TcState *s, CUtensorMap *map, const void *ptr, uint64_t inner, uint64_t rows,
                        uint32_t box_rows)
{
    cuuint64_t dims[2] = {inner, rows};
    cuuint64_t strides[1] = {inner};
    cuuint32_t box[2] = {128u, box_rows};
    cuuint32_t es[2] = {1, 1};
    return s->encode(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(ptr), dims, strides, box, es,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace mrp
