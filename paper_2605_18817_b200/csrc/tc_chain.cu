// The head chain for few activation rows as ONE persistent kernel (sm_100a, cooperative launch).
//
// For a handful of masked rows each GEMM of the chain (gate/up and down projection of every
// head, a1) moves 17-67 MB of weights and lasts a few microseconds; run as separate kernels
// they spend more time on launch, ring fill, first-use code fetch and drain than on the weights.
// Here the 2K GEMMs are phases of one kernel: every CTA walks the phases with the same TMA ring,
// MMA issuer and epilogue warps as the few-row kernels (tc_skinny.cu: weight rows on the MMA M
// axis, bf16 hi + lo activation rows stacked on N, one 128-row weight tile and one slice of the
// contraction per CTA and phase).  A phase needs the previous phase's activations, so the
// CTAs meet at a grid barrier between phases -- but the weights depend on nothing: the producer
// fills the ring with the next phase's weight tiles before it waits
// (three stages at once, the rest of the ring once the CTA has parked its own slice), and only
// the activation tiles are fetched after the barrier.
// A weight tile that is split over several CTAs is finished in three steps: every CTA parks its
// slice of the accumulator in scratch, the CTAs of the tile meet at a counter, and each finishes
// its share of the tile's output rows from the parked slices, added in slice order (so every SM
// takes part in the element-wise work, and the result does not depend on arrival order).  A
// gate/up tile that one CTA owns alone is finished straight from the accumulator.
// Every wait is bounded: a barrier or mbarrier wait that runs out sets MRP_DEV_TIMEOUT and the
// CTA leaves; the others then run out as well.
#include <cuda_fp16.h>
#include <string.h>

#include <atomic>

#include "tc_common.cuh"

namespace mrp {
namespace {

constexpr int kChThreads = 192;
constexpr int kChWTile = 128 * 128;
constexpr int kChAuxBytes = 20480;
constexpr int kChAuxRstd = 0;              // float[128]
constexpr int kChAuxVote = 768;            // int
constexpr int kChAuxReleased = 772;        // int: phases whose barrier this CTA has seen released
constexpr int kChAuxParked = 776;          // int: phases whose slice this CTA has parked (or had none to park)
constexpr int kChEarlyStages = 3;          // stages of the next phase fetched before the slice is parked
constexpr int kChAuxSq = 4096;             // float[4096]: squares of a share's outputs
constexpr int kChMaxShare = 4096;          // outputs a CTA finishes per down-projection phase, at most
constexpr int kChTilesPerPhase = 448;      // arrival counters per phase
constexpr int kChMaxPhases = 8;
constexpr long long kBarrierCycles = 1000000000LL;   // bound on a grid-barrier wait (about 0.5 s)

enum { CH_GU = 0, CH_DN = 1, CH_LIN = 2, CH_ATT = 3, CH_CAT = 4 };   // from LIN on: the module's phases (MOD instantiations)

constexpr int kModChainLayers = 4;     // module layers one launch can hold
constexpr int kModChainPhases = 2 + 5 * kModChainLayers;   // fusion rows + projection, five per layer
template <int NM>
struct ChainMapsT {
    CUtensorMap m[NM];
};
// head chain: 0: head input (xg), 1: SwiGLU output (act), 2+3h: gate, 3+3h: up, 4+3h: down of head h
using ChainMaps = ChainMapsT<2 + 3 * 4>;
// module step: 0 xa, 1 act, 2 xb, 3 [h ; emb] rows, 4 fusion projection, 5 + 7 l ...: q k v o gate up down of layer l
using ModChainMaps = ChainMapsT<5 + 7 * kModChainLayers>;

struct ChainPhase {
    int kind;
    int k_chunks;        // contraction extent / 64
    int n_tiles;         // 128-row weight tiles (GU: 64 gate + 64 up rows)
    int n_split;         // CTAs per tile, each a slice of the contraction
    int w_rows;          // weight rows (GU: gate rows)
    int map_x, map_w0, map_w1;
    int ssq_idx;         // GU: head index whose sums of squares normalise the input; DN: the one it adds to
    const __nv_bfloat16 *gamma_next;   // DN
    __nv_bfloat16 *xg_next;
    __nv_bfloat16 *xt_k;
    __half *xt16_k;
    float *hidden_out;
    // LIN (a plain product of the module): out[m, j] (+)= rstd(m) * sum, rstd from slot ssq_in of ssq_fix (< 0: 1);
    // with xg_next also out * gamma_next in operand form and the sums of squares of out added to slot ssq_idx.
    // lin3_tiles > 0: three matrices of lin3_tiles tiles each (maps map_w0, +1, +2; results lin_out, lin_out1, lin_out2)
    float *lin_out, *lin_out1, *lin_out2;
    int lin_acc, ssq_in, lin3_tiles;
    // ATT (no product): block-local attention over q, k, v [M, d] (fp32) into att_out in operand form
    const float *att_q, *att_k, *att_v;
    __nv_bfloat16 *att_out;
    int att_L, att_H;
    __nv_bfloat16 *att_pk, *att_pv;  // the layer's clean-prefix cache [*, H, pcap, dh] (nullptr: block-local attention)
    int zero_slot0, zero_slot1;      // ssq_fix slots this phase clears for later phases of the launch (< 0: none)
    int fin;                         // LIN that completes Delta: its finish also does h <- h + Delta and the LM-head operand
};

// What the module's first phase (CAT: the rows [h ; emb[x]] in operand form) and the finish of its last product
// (h <- h + Delta and the LM-head operand of the masked rows) need.
struct ModEnds {
    const int32_t *tokens;
    const __nv_bfloat16 *hidden0, *emb;
    float *h_state, *z;
    __nv_bfloat16 *cat;
    int first_step, mask_token, emb_rows;
    const int32_t *row_index;
    int n_masked;
    __nv_bfloat16 *xt;       // LM-head operand rows (step 0 zero rows, then h - h_0), lo rows lo_xt rows further on
    __half *xt16;
    float *hidden_out;
    const int32_t *plen;     // clean prefix: rows in use per sequence, rows per slab, whether the block's own keys and
    int pcap, append;        // values are stored behind them
    int att_nch, att_gpc;    // ... chunks of the key range per (block, head), groups of 32 keys per chunk
    int att_mma;             // ... the prefix chunks as tensor-core products, the block's keys a chunk of their own
    float *att_part;         // partial results of the chunks
    int *att_counters;       // arrivals per (block, head): zero before and after the launch
};

template <int NP>
struct ChainParamsT {
    int n_phases, n_stages, tmem_cols;
    int M, d, F, n_rs;
    int lo_x, lo_xt;         // row offset of the lo block in the head operands / the LM-head operand
    float eps;
    ChainPhase ph[NP];
    ModEnds mod;
    __nv_bfloat16 *act;
    float *hcur;
    const float *h0f;
    unsigned long long *ssq_fix;   // [5][128] sums of squares in 2^-24 fixed point: integer adds commute,
                                   // so the CTAs of a phase can add their shares in any order
    float *scratch;          // partial accumulators [cta][RP][128]
    int32_t *counters;       // arrivals per (phase, tile) (zero at launch)
    unsigned int *grid_bar;  // CTAs that have finished a phase, summed over phases (zero at launch)
    int32_t *status;
    int32_t *user_status;
};
static_assert(kModChainBarInts == kModChainPhases * kChTilesPerPhase + 1, "counter array of the one-launch module step");
using ChainParams = ChainParamsT<kChMaxPhases>;
using ModChainParams = ChainParamsT<kModChainPhases>;
template <bool MOD> struct ChainTypes { using Maps = ChainMaps; using Params = ChainParams; };
template <> struct ChainTypes<true> { using Maps = ModChainMaps; using Params = ModChainParams; };

__device__ __forceinline__ void ch_epi_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
__device__ __forceinline__ void ch_store_hi_lo(__nv_bfloat16 *dst, size_t lo_off, float v)
{
    const __nv_bfloat16 hi = __float2bfloat16_rn(v);
    dst[0] = hi;
    dst[lo_off] = __float2bfloat16_rn(v - __bfloat162float(hi));
}
// four consecutive values as bf16 hi + lo pairs, one 8-byte store each
__device__ __forceinline__ void ch_store_split4(__nv_bfloat16 *dst, size_t lo_off, const float *v)
{
    uint32_t hi[2], lo[2];
    split_bf16(v[0], v[1], hi[0], lo[0]);
    split_bf16(v[2], v[3], hi[1], lo[1]);
    *reinterpret_cast<uint2 *>(dst) = make_uint2(hi[0], hi[1]);
    *reinterpret_cast<uint2 *>(dst + lo_off) = make_uint2(lo[0], lo[1]);
}
__device__ __forceinline__ unsigned int ld_acquire_u32(const unsigned int *p)
{
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// Waits until `target` arrivals have been counted; false if the wait ran out or another role gave up.
template <typename P>
__device__ __forceinline__ bool grid_bar_wait(const unsigned int *bar, unsigned int target, volatile int *abort_flag,
                                              const P &p)
{
    if ((int)(ld_acquire_u32(bar) - target) >= 0) return true;
    const long long t0 = clock64();
    while ((int)(ld_acquire_u32(bar) - target) < 0) {
        __nanosleep(128);
        if (*abort_flag) return false;
        if (clock64() - t0 > kBarrierCycles) {
            *abort_flag = 1;
            atomicOr(p.status, MRP_DEV_TIMEOUT);
            if (p.user_status) atomicOr(p.user_status, MRP_DEV_TIMEOUT);
            return false;
        }
    }
    return true;
}

// MOD: the instantiation that also knows the module's phase kinds (LIN, ATT); the head chain's own instantiations
// compile none of that code.
template <int RP, int KC, bool MOD = false>
__global__ void __launch_bounds__(kChThreads, 1)
sk_chain_kernel(const __grid_constant__ typename ChainTypes<MOD>::Maps maps,
                const __grid_constant__ typename ChainTypes<MOD>::Params p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    constexpr int x_bytes = 2 * RP * 128;            // hi rows then lo rows of one k-chunk
    constexpr int sub_bytes = kChWTile + x_bytes;     // one k-chunk: weight tile, then activation rows
    constexpr int stage_bytes = KC * sub_bytes;       // a ring stage holds KC k-chunks: one barrier wait and
                                                      // one commit per 4 * KC MMAs
    const uint32_t bars = base + (uint32_t)p.n_stages * stage_bytes;
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (p.n_stages + s); };
    auto tfull_bar = [&](int a) { return bars + 8u * (2 * p.n_stages + a); };
    auto tempty_bar = [&](int a) { return bars + 8u * (2 * p.n_stages + 2 + a); };
    uint8_t *gen_base = smem_raw + (base - smem_u32(smem_raw));
    uint8_t *after_bars = gen_base + (size_t)p.n_stages * stage_bytes + 8 * (2 * p.n_stages + 4);
    uint32_t *tmem_holder = reinterpret_cast<uint32_t *>(after_bars);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_holder + 1);
    uint8_t *aux = after_bars + 16;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int cta = blockIdx.x, G = gridDim.x;

    // this CTA's share of phase i: weight tile, chunk range; false if it has none
    auto share = [&](int i, int &tile, int &kc0, int &nk) {
        const ChainPhase &ph = p.ph[i];
        if (cta >= ph.n_tiles * ph.n_split) return false;
        const int cps = (ph.k_chunks + ph.n_split - 1) / ph.n_split;
        tile = cta / ph.n_split;
        kc0 = (cta % ph.n_split) * cps;
        nk = min(ph.k_chunks, kc0 + cps) - kc0;
        return true;
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.n_stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 4); }
        *abort_flag = 0;
        *reinterpret_cast<volatile int *>(aux + kChAuxParked) = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        prefetch_tmap(&maps.m[0]);
        prefetch_tmap(&maps.m[2]);
        prefetch_tmap(&maps.m[3]);
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
    pdl_trigger();

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            const uint64_t pol_w = l2_policy_evict_first(), pol_x = l2_policy_evict_last();
            int it = 0;                       // chunks issued so far, over all phases
            bool ok = true;
            for (int i = 0; i < p.n_phases && ok; ++i) {
                int tile, kc0, nk;
                if (!share(i, tile, kc0, nk)) continue;
                const ChainPhase &ph = p.ph[i];
                auto stage_of = [&](int n) { return n % p.n_stages; };
                auto claim = [&](int n) {     // wait until the stage of chunk n is free, arm its barrier
                    const int s = stage_of(n), use = n / p.n_stages;
                    if (use > 0 && !mbar_wait(empty_bar(s), (uint32_t)((use - 1) & 1), abort_flag, p)) return false;
                    mbar_expect_tx(full_bar(s), (uint32_t)stage_bytes);
                    return true;
                };
                auto load_w = [&](int n, int kk) {
#pragma unroll
                    for (int b = 0; b < KC; ++b) {
                        const uint32_t sw = base + (uint32_t)stage_of(n) * stage_bytes + b * sub_bytes;
                        const int col = (kc0 + kk * KC + b) * kBK;
                        if (ph.kind == CH_GU) {
                            tma_load_2d_hint(sw, &maps.m[ph.map_w0], col, tile * 64, full_bar(stage_of(n)), pol_w);
                            tma_load_2d_hint(sw + 64 * 128, &maps.m[ph.map_w1], col, tile * 64, full_bar(stage_of(n)), pol_w);
                        } else if (MOD && ph.kind == CH_LIN && ph.lin3_tiles > 0) {
                            const int which = tile / ph.lin3_tiles;
                            tma_load_2d_hint(sw, &maps.m[ph.map_w0 + which], col, (tile - which * ph.lin3_tiles) * 128,
                                             full_bar(stage_of(n)), pol_w);
                        } else {
                            tma_load_2d_hint(sw, &maps.m[ph.map_w0], col, tile * 128, full_bar(stage_of(n)), pol_w);
                        }
                    }
                };
                auto load_x = [&](int n, int kk) {
#pragma unroll
                    for (int b = 0; b < KC; ++b) {
                        const uint32_t sx = base + (uint32_t)stage_of(n) * stage_bytes + b * sub_bytes + kChWTile;
                        // one box: RP hi rows, then (the lo block starts at row RP of the buffer) RP lo rows
                        tma_load_2d_hint(sx, &maps.m[ph.map_x], (kc0 + kk * KC + b) * kBK, 0, full_bar(stage_of(n)), pol_x);
                    }
                };
                nk /= KC;                     // ring steps of this slice (KC divides every slice)
                // weights depend on nothing: put as many chunks of them in flight as the ring holds
                // The first few stages go out at once, so that the phase can start the moment its
                // activations exist; the rest of the ring waits until this CTA has parked the previous
                // phase's slice: those stores and their fence are on the critical path and take two
                // to four times as long while 20 MB of prefetch hit the memory system together.
                const int pre = min(p.n_stages, nk);
                for (int kk = 0; kk < pre && ok; ++kk) {
                    if (kk == kChEarlyStages && i > 0) {
                        volatile int *parked_s = reinterpret_cast<volatile int *>(aux + kChAuxParked);
                        const long long t0 = clock64();
                        while (*parked_s < i) {
                            if (*abort_flag || clock64() - t0 > 2 * kBarrierCycles) { ok = false; break; }
                        }
                        if (!ok) break;
                    }
                    ok = claim(it + kk);
                    if (ok) load_w(it + kk, kk);
                }
                if (!ok) break;
                // the activations are the previous phase's (or the previous kernel's) output
                if (i == 0) {
                    pdl_wait();
                } else {
                    // one thread of the CTA (epilogue thread 0) polls the grid barrier; wait for its word
                    volatile int *released_s = reinterpret_cast<volatile int *>(aux + kChAuxReleased);
                    const long long t0 = clock64();
                    bool passed = true;
                    while (*released_s < i) {
                        if (*abort_flag || clock64() - t0 > 2 * kBarrierCycles) { passed = false; break; }
                    }
                    if (!passed) break;
                }
                asm volatile("fence.proxy.async;" ::: "memory");
                for (int kk = 0; kk < pre; ++kk) load_x(it + kk, kk);
                for (int kk = pre; kk < nk && ok; ++kk) {
                    ok = claim(it + kk);
                    if (ok) { load_w(it + kk, kk); load_x(it + kk, kk); }
                }
                it += nk;
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        // The whole warp walks the loop (all values are warp-uniform); the elected lane issues.
        const uint32_t idesc = make_idesc(2 * RP);
        int n_acc = 0;
        int s = 0;                        // ring stage and its barrier phase, advanced chunk by chunk
        uint32_t ph_bit = 0;
        bool ok = true;
        for (int i = 0; i < p.n_phases && ok; ++i) {
            int tile, kc0, nk;
            if (!share(i, tile, kc0, nk)) continue;
            const int acc = n_acc & 1, use = n_acc >> 1;
            if (use > 0) ok = __all_sync(0xffffffffu, mbar_wait(tempty_bar(acc), (uint32_t)((use - 1) & 1), abort_flag, p));
            if (!ok) break;
            tc_fence_after();
            const uint32_t dt = __shfl_sync(0xffffffffu, tmem_base, 0) + (uint32_t)(acc * 2 * RP);
            nk /= KC;
            for (int kk = 0; kk < nk; ++kk) {
                const uint32_t sw = base + (uint32_t)s * stage_bytes;
                const uint32_t later = kk > 0 ? 1u : 0u;
                ok = __all_sync(0xffffffffu, mbar_wait(full_bar(s), ph_bit, abort_flag, p));
                if (!ok) break;
                tc_fence_after();
                if (elect_one()) {
#pragma unroll
                    for (int b = 0; b < KC; ++b) {
                        const uint64_t dw = make_smem_desc(sw + b * sub_bytes);
                        const uint64_t dx = make_smem_desc(sw + b * sub_bytes + kChWTile);
#pragma unroll
                        for (int k4 = 0; k4 < kBK / 16; ++k4)
                            umma_bf16(dt, dw + 2u * k4, dx + 2u * k4, idesc, (b > 0 || k4 > 0) ? 1u : later);
                    }
                    umma_commit(empty_bar(s));
                }
                __syncwarp();
                if (++s == p.n_stages) { s = 0; ph_bit ^= 1u; }
            }
            if (!ok) break;
            if (elect_one()) umma_commit(tfull_bar(acc));
            __syncwarp();
            ++n_acc;
        }
    } else {
        // ---------------- epilogue warps ----------------
        // Per phase: (1) thread t parks TMEM lane t (weight row t of the tile) of this slice's
        // accumulator in global scratch; (2) the CTAs of the tile wait for one another; (3) every
        // CTA finishes its own share of the tile's rows from the parked slices, added in slice
        // order, so all SMs take part in the element-wise work and its memory round trips.
        const int q = warp & 3;
        const int t = q * 32 + lane;
        const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16);
        float *rstd_s = reinterpret_cast<float *>(aux + kChAuxRstd);
        float *sq_s = reinterpret_cast<float *>(aux + kChAuxSq);
        volatile int *vote_s = reinterpret_cast<volatile int *>(aux + kChAuxVote);
        volatile int *released_s = reinterpret_cast<volatile int *>(aux + kChAuxReleased);
        const int n_ch = (p.M + 15) >> 4;
        int n_acc = 0;
        bool alive = true;
        // row m of the LM-head operand: zero rows of step 0, then h - h_0 (hi + lo; fp16 copy where that LM head runs)
        auto fin_put = [&](int m, int j, float h, float r) {
            const ModEnds &e = p.mod;
            const size_t o = (size_t)m * p.d + j;
            if (e.hidden_out) e.hidden_out[o] = h;
            e.xt[o] = __float2bfloat16(0.f);
            e.xt[(size_t)p.lo_xt * p.d + o] = __float2bfloat16(0.f);
            ch_store_hi_lo(e.xt + (size_t)e.n_masked * p.d + o, (size_t)p.lo_xt * p.d, r);
            if (e.xt16) e.xt16[o] = __float2half_rn(r);
        };
        pdl_wait();
        for (int i = 0; i < p.n_phases && alive; ++i) {
            const ChainPhase &ph = p.ph[i];
            // everything this phase reads was written before the previous phase's barrier
            if (t == 0) {
                if (i == 0) { *vote_s = 0; *released_s = 0; }
                else if (grid_bar_wait(p.grid_bar, (unsigned int)i * G, abort_flag, p)) *released_s = i;
                else *vote_s = 1;
            }
            ch_epi_sync();
            if (*vote_s == 1) { alive = false; break; }
            if (MOD && ph.fin) {
                // the product that completes Delta: dense position -> masked row (or -1), for its finish below
                // (the buffer of squares is free: no norm follows this product)
                const ModEnds &e = p.mod;
                int *inv = reinterpret_cast<int *>(sq_s);
                for (int i2 = t; i2 < p.M; i2 += 128) inv[i2] = -1;
                ch_epi_sync();
                if (t == 0) {
                    for (int m = 0; m < e.n_masked; ++m) {
                        const int idx = e.row_index ? e.row_index[m] : m;
                        if (row_ok(idx, p.M)) inv[idx] = m;
                        else if (cta == 0) {
                            atomicOr(p.status, MRP_DEV_BAD_INDEX);
                            if (p.user_status) atomicOr(p.user_status, MRP_DEV_BAD_INDEX);
                        }
                    }
                }
                ch_epi_sync();
            }
            int tile, kc0, nk;
            const bool active = share(i, tile, kc0, nk);
            if (active) {
                const int split = cta % ph.n_split;
                if (ph.kind == CH_GU) {
                    if (t < p.M) {
                        const unsigned long long v = __ldcg(p.ssq_fix + ph.ssq_idx * 128 + t);
                        const float s = (float)((double)v * (1.0 / 16777216.0));
                        rstd_s[t] = rsqrtf(s / (float)p.d + p.eps);
                    }
                }
                if (MOD && ph.kind == CH_LIN) {
                    if (t < p.M) {
                        float r = 1.f;
                        if (ph.ssq_in >= 0) {
                            const unsigned long long v = __ldcg(p.ssq_fix + ph.ssq_in * 128 + t);
                            r = rsqrtf((float)((double)v * (1.0 / 16777216.0)) / (float)p.d + p.eps);
                        }
                        rstd_s[t] = r;
                    }
                }
                const int acc = n_acc & 1, use = n_acc >> 1;
                ++n_acc;
                const uint32_t lane_addr = lane_base + (uint32_t)(acc * 2 * RP);
                bool ok = __all_sync(0xffffffffu, mbar_wait(tfull_bar(acc), (uint32_t)(use & 1), abort_flag, p));
                if (!ok && lane == 0) *vote_s = 1;
                ch_epi_sync();                      // also publishes rstd_s
                if (*vote_s == 1) { alive = false; break; }
                tc_fence_after();
                if (ph.kind == CH_GU && ph.n_split == 1) {
                    // The tile is this CTA's alone: no slices to add, so the outputs are finished straight
                    // from the accumulator.  Gate row c and up row c of an output sit in lanes c and c + 64:
                    // they meet through shared memory, 16 batch rows at a time.
                    float *exch = sq_s;                              // [16][128]
#pragma unroll 1
                    for (int ch = 0; ch < n_ch; ++ch) {
                        float v[16], w[16];
                        tmem_ld16(lane_addr + ch * 16, v);
                        tmem_ld16(lane_addr + RP + ch * 16, w);
#pragma unroll
                        for (int j = 0; j < 16; ++j) exch[j * 128 + t] = v[j] + w[j];
                        ch_epi_sync();
                        // thread = (batch row j of the 16, 8 consecutive outputs): two 16-byte stores
                        const int j = t >> 3, c0 = (t & 7) * 8, m = ch * 16 + j, f0 = tile * 64 + c0;
                        if (m < p.M && f0 < ph.w_rows) {
                            const float4 *gp = reinterpret_cast<const float4 *>(exch + j * 128 + c0);
                            const float4 *up = reinterpret_cast<const float4 *>(exch + j * 128 + 64 + c0);
                            const float4 g0 = gp[0], g1 = gp[1], u0 = up[0], u1 = up[1];
                            const float gg[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
                            const float uu[8] = {u0.x, u0.y, u0.z, u0.w, u1.x, u1.y, u1.z, u1.w};
                            const float rs = rstd_s[m];
                            float av[8];
#pragma unroll
                            for (int q = 0; q < 8; ++q) {
                                const float g = gg[q] * rs;
                                av[q] = g / (1.f + __expf(-g)) * (uu[q] * rs);
                            }
                            store_split<8>(p.act + (size_t)m * p.F + f0, (size_t)p.lo_x * p.F, av);
                        }
                        ch_epi_sync();
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(tempty_bar(acc));     // the accumulator buffer is free again
                } else {
                    // (1) park this slice: scratch[cta][column][lane]
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
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(tempty_bar(acc));     // the accumulator buffer is free again
                    // (2) meet the other CTAs of the tile.  One thread's fence after the CTA barrier publishes
                    // every thread's stores (fences are cumulative), and costs one wait instead of four.
                    ch_epi_sync();
                    if (t == 0) {
                        __threadfence();
                        *reinterpret_cast<volatile int *>(aux + kChAuxParked) = i + 1;
                        unsigned int *cnt = reinterpret_cast<unsigned int *>(p.counters) + i * kChTilesPerPhase + tile;
                        atomicAdd(cnt, 1u);
                        if (!grid_bar_wait(cnt, (unsigned int)ph.n_split, abort_flag, p)) *vote_s = 1;
                    }
                    ch_epi_sync();
                    if (*vote_s == 1) { alive = false; break; }
                    // (3) this CTA's share of the tile's output rows, element by element from the parked slices
                    const int rows_tile = ph.kind == CH_GU ? 64 : 128;
                    const int per = (rows_tile + ph.n_split - 1) / ph.n_split;
                    const int r0 = split * per;
                    const int n_r = max(0, min(rows_tile, r0 + per) - r0);
                    const int n_items = n_r * p.M;
                    const float *first = p.scratch + ((size_t)tile * ph.n_split * RP) * 128;
                    if (ph.kind == CH_GU) {
                        bool done = false;
                        if constexpr (RP >= 32) {
                            // many batch rows: four consecutive outputs per item, 16-byte loads, 8-byte stores
                            if ((per & 3) == 0 && (ph.w_rows & 3) == 0 && n_r > 0) {
                                const int n_g = n_r >> 2;
                                done = true;
#pragma unroll 2
                                for (int e = t; e < n_g * p.M; e += 128) {
                                    const int m = e / n_g, row = r0 + ((e - m * n_g) << 2);
                                    const int f = tile * 64 + row;
                                    if (f < ph.w_rows) {
                                        float4 g = make_float4(0.f, 0.f, 0.f, 0.f), u = g;
                                        for (int s0 = 0; s0 < ph.n_split; s0 += 4) {  // slice order; 4 slices' loads in flight
                                            float4 gs[4], us[4];
#pragma unroll
                                            for (int k = 0; k < 4; ++k) {
                                                const float *src = first + ((size_t)(s0 + k) * RP + m) * 128 + row;
                                                const bool in = s0 + k < ph.n_split;
                                                gs[k] = in ? __ldcg(reinterpret_cast<const float4 *>(src)) : make_float4(0.f, 0.f, 0.f, 0.f);
                                                us[k] = in ? __ldcg(reinterpret_cast<const float4 *>(src + 64)) : make_float4(0.f, 0.f, 0.f, 0.f);
                                            }
#pragma unroll
                                            for (int k = 0; k < 4; ++k) {
                                                g.x += gs[k].x; g.y += gs[k].y; g.z += gs[k].z; g.w += gs[k].w;
                                                u.x += us[k].x; u.y += us[k].y; u.z += us[k].z; u.w += us[k].w;
                                            }
                                        }
                                        const float rs = rstd_s[m];
                                        const float gg[4] = {g.x * rs, g.y * rs, g.z * rs, g.w * rs};
                                        const float uu[4] = {u.x * rs, u.y * rs, u.z * rs, u.w * rs};
                                        float av[4];
#pragma unroll
                                        for (int k = 0; k < 4; ++k) av[k] = gg[k] / (1.f + __expf(-gg[k])) * uu[k];
                                        ch_store_split4(p.act + (size_t)m * p.F + f, (size_t)p.lo_x * p.F, av);
                                    }
                                }
                            }
                        }
                        if (!done) {
#pragma unroll 2
                            for (int e = t; e < n_items; e += 128) {
                                const int m = e / n_r, row = r0 + (e - m * n_r);
                                const int f = tile * 64 + row;
                                if (f < ph.w_rows) {
                                    float g = 0.f, u = 0.f;
                                    for (int s0 = 0; s0 < ph.n_split; s0 += 8) {  // slice order; 8 slices' loads in flight
                                        float gs[8], us[8];
#pragma unroll
                                        for (int k = 0; k < 8; ++k) {
                                            const float *src = first + ((size_t)(s0 + k) * RP + m) * 128 + row;
                                            gs[k] = (s0 + k < ph.n_split) ? __ldcg(src) : 0.f;
                                            us[k] = (s0 + k < ph.n_split) ? __ldcg(src + 64) : 0.f;
                                        }
#pragma unroll
                                        for (int k = 0; k < 8; ++k) { g += gs[k]; u += us[k]; }
                                    }
                                    g *= rstd_s[m];
                                    u *= rstd_s[m];
                                    ch_store_hi_lo(p.act + (size_t)m * p.F + f, (size_t)p.lo_x * p.F, g / (1.f + __expf(-g)) * u);
                                }
                            }
                        }
                    } else if (MOD && ph.kind == CH_LIN) {
                        // a plain product: this CTA's rows of the tile, one output at a time from the parked slices
                        const int which = ph.lin3_tiles > 0 ? tile / ph.lin3_tiles : 0;
                        const int tile_w = ph.lin3_tiles > 0 ? tile - which * ph.lin3_tiles : tile;
                        float *dst = which == 0 ? ph.lin_out : which == 1 ? ph.lin_out1 : ph.lin_out2;
#pragma unroll 2
                        for (int e = t; e < n_items; e += 128) {
                            const int m = e / n_r, row = r0 + (e - m * n_r);
                            const int j = tile_w * 128 + row;
                            float sq = 0.f;
                            if (j < ph.w_rows) {
                                const size_t o = (size_t)m * ph.w_rows + j;
                                float a = 0.f;
                                for (int s0 = 0; s0 < ph.n_split; s0 += 8) {      // slice order; 8 slices' loads in flight
                                    float as[8];
#pragma unroll
                                    for (int k = 0; k < 8; ++k)
                                        as[k] = (s0 + k < ph.n_split) ? __ldcg(first + ((size_t)(s0 + k) * RP + m) * 128 + row) : 0.f;
#pragma unroll
                                    for (int k = 0; k < 8; ++k) a += as[k];
                                }
                                float h = a * rstd_s[m];
                                if (ph.lin_acc) h += __ldcg(dst + o);
                                dst[o] = h;
                                sq = h * h;
                                if (ph.fin) {
                                    // Delta is complete here: h <- h + Delta, and the LM-head operand of a masked position
                                    const ModEnds &en = p.mod;
                                    const int *inv = reinterpret_cast<const int *>(sq_s);
                                    const float hs = __ldcg(en.h_state + o) + h;
                                    en.h_state[o] = hs;
                                    if (inv[m] >= 0) fin_put(inv[m], j, hs, hs - __bfloat162float(en.hidden0[o]));
                                }
                                if (ph.xg_next) ch_store_hi_lo(ph.xg_next + o, (size_t)p.lo_x * ph.w_rows, h * __bfloat162float(ph.gamma_next[j]));
                            }
                            if (ph.xg_next) sq_s[e] = sq;        // (a share without a norm behind it may exceed the buffer)
                        }
                        if (ph.xg_next) {
                            ch_epi_sync();
                            for (int m = t; m < p.M; m += 128) {
                                float s2 = 0.f;
                                for (int r = 0; r < n_r; ++r) s2 += sq_s[m * n_r + r];
                                atomicAdd(p.ssq_fix + ph.ssq_idx * 128 + m, (unsigned long long)__double2ll_rn((double)s2 * 16777216.0));
                            }
                        }
                    } else {
                        int n_sq = n_r;                      // entries of the buffer of squares per batch row
                        bool done = false;
                        if constexpr (RP >= 32) {
                            // Many batch rows: a share is thousands of outputs, so four consecutive output
                            // rows are handled per item with 16-byte loads and 8-byte stores.
                            if ((per & 3) == 0 && (ph.w_rows & 3) == 0 && n_r > 0) {
                                const int n_g = n_r >> 2;
                                n_sq = n_g;
                                done = true;
#pragma unroll 2
                                for (int e = t; e < n_g * p.M; e += 128) {
                                    const int m = e / n_g, row = r0 + ((e - m * n_g) << 2);
                                    const int j = tile * 128 + row;
                                    float sq = 0.f;
                                    if (j < ph.w_rows) {
                                        const size_t o = (size_t)m * p.d + j;
                                        const float4 hc = __ldcg(reinterpret_cast<const float4 *>(p.hcur + o));
                                        const float4 h0 = __ldg(reinterpret_cast<const float4 *>(p.h0f + o));
                                        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
                                        for (int s0 = 0; s0 < ph.n_split; s0 += 8) {  // slice order; 8 slices' loads in flight
                                            float4 as[8];
#pragma unroll
                                            for (int k = 0; k < 8; ++k)
                                                as[k] = (s0 + k < ph.n_split)
                                                            ? __ldcg(reinterpret_cast<const float4 *>(first + ((size_t)(s0 + k) * RP + m) * 128 + row))
                                                            : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                                            for (int k = 0; k < 8; ++k) { a.x += as[k].x; a.y += as[k].y; a.z += as[k].z; a.w += as[k].w; }
                                        }
                                        const float h[4] = {hc.x + a.x, hc.y + a.y, hc.z + a.z, hc.w + a.w};
                                        const float hz[4] = {h0.x, h0.y, h0.z, h0.w};
                                        *reinterpret_cast<float4 *>(p.hcur + o) = make_float4(h[0], h[1], h[2], h[3]);
                                        if (ph.hidden_out) *reinterpret_cast<float4 *>(ph.hidden_out + o) = make_float4(h[0], h[1], h[2], h[3]);
                                        sq = (h[0] * h[0] + h[1] * h[1]) + (h[2] * h[2] + h[3] * h[3]);
                                        float r[4], xn[4];
#pragma unroll
                                        for (int k = 0; k < 4; ++k) {
                                            r[k] = h[k] - hz[k];
                                            xn[k] = ph.xg_next ? h[k] * __bfloat162float(ph.gamma_next[j + k]) : 0.f;
                                        }
                                        ch_store_split4(ph.xt_k + o, (size_t)p.lo_xt * p.d, r);
                                        if (ph.xt16_k) {
                                            __half2 hh[2] = {__floats2half2_rn(r[0], r[1]), __floats2half2_rn(r[2], r[3])};
                                            *reinterpret_cast<uint2 *>(ph.xt16_k + o) = *reinterpret_cast<uint2 *>(hh);
                                        }
                                        if (ph.xg_next) ch_store_split4(ph.xg_next + o, (size_t)p.lo_x * p.d, xn);
                                    }
                                    sq_s[e] = sq;
                                }
                            }
                        }
                        if (!done) {
#pragma unroll 2
                            for (int e = t; e < n_items; e += 128) {
                                const int m = e / n_r, row = r0 + (e - m * n_r);
                                const int j = tile * 128 + row;
                                float sq = 0.f;
                                if (j < ph.w_rows) {
                                    const size_t o = (size_t)m * p.d + j;
                                    const float hc = __ldcg(p.hcur + o), h0 = __ldg(p.h0f + o);
                                    float a = 0.f;
                                    for (int s0 = 0; s0 < ph.n_split; s0 += 8) {  // slice order; 8 slices' loads in flight
                                        float as[8];
#pragma unroll
                                        for (int k = 0; k < 8; ++k)
                                            as[k] = (s0 + k < ph.n_split) ? __ldcg(first + ((size_t)(s0 + k) * RP + m) * 128 + row) : 0.f;
#pragma unroll
                                        for (int k = 0; k < 8; ++k) a += as[k];
                                    }
                                    const float h = hc + a;
                                    p.hcur[o] = h;
                                    if (ph.hidden_out) ph.hidden_out[o] = h;
                                    sq = h * h;
                                    ch_store_hi_lo(ph.xt_k + o, (size_t)p.lo_xt * p.d, h - h0);
                                    if (ph.xt16_k) ph.xt16_k[o] = __float2half_rn(h - h0);
                                    if (ph.xg_next) ch_store_hi_lo(ph.xg_next + o, (size_t)p.lo_x * p.d, h * __bfloat162float(ph.gamma_next[j]));
                                }
                                sq_s[e] = sq;
                            }
                        }
                        ch_epi_sync();
                        // this CTA's rows, in row order, then one integer add per row of the batch
                        for (int m = t; m < p.M; m += 128) {
                            float s = 0.f;
                            for (int r = 0; r < n_sq; ++r) s += sq_s[m * n_sq + r];
                            atomicAdd(p.ssq_fix + ph.ssq_idx * 128 + m,
                                      (unsigned long long)__double2ll_rn((double)s * 16777216.0));
                        }
                    }
                }
            }
            if (MOD) {
                if (cta == 0 && t < p.M) {          // sums of squares later phases of this launch add to start at zero
                    if (ph.zero_slot0 >= 0) p.ssq_fix[ph.zero_slot0 * 128 + t] = 0ull;
                    if (ph.zero_slot1 >= 0) p.ssq_fix[ph.zero_slot1 * 128 + t] = 0ull;
                }
                if (ph.kind == CH_CAT) {
                    // the rows [h_i ; emb[x_i]] in operand form; on the first step of a backbone forward h is the
                    // backbone's hidden state, which also starts the running state
                    const ModEnds &e = p.mod;
                    const int d2 = 2 * p.d;
                    for (int idx = cta * 128 + t; idx < p.M * p.d; idx += G * 128) {
                        const int pos = idx / p.d, j = idx - pos * p.d;
                        int tok = e.tokens[pos];
                        if (tok >= e.emb_rows || tok < -1) {          // outside the table: reads as masked, raises the bit
                            if (j == 0) {
                                atomicOr(p.status, MRP_DEV_BAD_INDEX);
                                if (p.user_status) atomicOr(p.user_status, MRP_DEV_BAD_INDEX);
                            }
                            tok = -1;
                        }
                        if (tok < 0) tok = e.mask_token;
                        const float h = e.first_step ? __bfloat162float(e.hidden0[idx]) : __ldcg(e.h_state + idx);
                        if (e.first_step) e.h_state[idx] = h;
                        ch_store_hi_lo(e.cat + (size_t)pos * d2 + j, (size_t)p.lo_x * d2, h);
                        e.cat[(size_t)pos * d2 + p.d + j] = e.emb[(size_t)tok * p.d + j];       // a bf16 value: no remainder
                        e.cat[((size_t)p.lo_x + pos) * d2 + p.d + j] = __float2bfloat16(0.f);
                    }
                }
                if (ph.kind == CH_LIN && ph.fin) {
                    // masked rows whose index is out of range, or names a position that a later row names too: zero rows
                    const ModEnds &e = p.mod;
                    const int *inv = reinterpret_cast<const int *>(sq_s);
                    for (int m = 0; m < e.n_masked; ++m) {
                        const int idx = e.row_index ? e.row_index[m] : m;
                        if (!row_ok(idx, p.M) || inv[idx] != m)
                            for (int j = cta * 128 + t; j < p.d; j += G * 128) fin_put(m, j, 0.f, 0.f);
                    }
                }
                if (ph.kind == CH_ATT && ph.att_pk) {
                    // attention behind a clean prefix: the four warps on one (block, attention head, chunk of the keys)
                    // at a time; the CTA that arrives last at a (block, head) merges its chunks
                    const ModEnds &e = p.mod;
                    const int L = ph.att_L, H = ph.att_H, dh = p.d / H, n_ch = e.att_nch;
                    for (int unit = cta; unit < (p.M / L) * H * n_ch; unit += G) {
                        const int ch = unit % n_ch, bh = unit / n_ch, b = bh / H, hd = bh - b * H;
                        int P = e.plen[b];
                        bool bad = P < 0 || P > e.pcap;
                        P = P < 0 ? 0 : (P > e.pcap ? e.pcap : P);
                        const bool store = e.append && !bad && P + L <= e.pcap;
                        bad = bad || (e.append && !store);
                        if (bad && t == 0 && hd == 0 && ch == 0) {
                            atomicOr(p.status, MRP_DEV_BAD_INDEX);
                            if (p.user_status) atomicOr(p.user_status, MRP_DEV_BAD_INDEX);
                        }
                        const size_t head = (size_t)hd * dh, slab = ((size_t)b * H + hd) * e.pcap * dh, blk = (size_t)b * L * p.d + head;
                        if (store && ch == 0) {       // rows this call never reads
                            for (int x = t; x < L * dh; x += 128) {
                                const int i2 = x / dh, cidx = x - i2 * dh;
                                ph.att_pk[slab + (size_t)(P + i2) * dh + cidx] = __float2bfloat16_rn(__ldcg(ph.att_k + blk + (size_t)i2 * p.d + cidx));
                                ph.att_pv[slab + (size_t)(P + i2) * dh + cidx] = __float2bfloat16_rn(__ldcg(ph.att_v + blk + (size_t)i2 * p.d + cidx));
                            }
                        }
                        att_unit<__nv_bfloat16, true>(ph.att_q + blk, ph.att_pk + slab, ph.att_pv + slab, P, ph.att_k + blk, ph.att_v + blk, L, p.d,
                                                dh, ch, n_ch, e.att_gpc, e.att_mma, e.att_part + (size_t)bh * n_ch * L * (dh + 2), e.att_counters + bh,
                                                sq_s, q, lane, [&] { ch_epi_sync(); }, [&](int i2, int cidx, float val) {
                                                    ch_store_hi_lo(ph.att_out + blk + (size_t)i2 * p.d + cidx, (size_t)p.lo_x * p.d, val);
                                                });
                    }
                } else if (ph.kind == CH_ATT) {
                    // block-local bidirectional attention, a warp per (position, attention head) over the whole grid;
                    // lanes over the head's features, one warp sum per key; output in operand form (hi + lo)
                    const int L = ph.att_L, H = ph.att_H, dh = p.d / H;
                    const float scale = rsqrtf((float)dh);
                    for (int item = cta * 4 + q; item < p.M * H; item += G * 4) {
                        const int pos = item / H, hd = item - pos * H, b0 = (pos / L) * L;
                        const float *qi = ph.att_q + (size_t)pos * p.d + (size_t)hd * dh;
                        // online softmax over the keys of the block: running maximum, sum and output
                        float mx = -INFINITY, sum = 0.f;
                        float oacc[8];                   // dh <= 256: eight features per lane at most
#pragma unroll
                        for (int u = 0; u < 8; ++u) oacc[u] = 0.f;
                        for (int j = 0; j < L; ++j) {
                            const float *kj = ph.att_k + (size_t)(b0 + j) * p.d + (size_t)hd * dh;
                            const float *vj = ph.att_v + (size_t)(b0 + j) * p.d + (size_t)hd * dh;
                            float sd = 0.f;
                            for (int cidx = lane; cidx < dh; cidx += 32) sd = fmaf(__ldcg(qi + cidx), __ldcg(kj + cidx), sd);
#pragma unroll
                            for (int o2 = 16; o2 > 0; o2 >>= 1) sd += __shfl_xor_sync(0xffffffffu, sd, o2);
                            sd *= scale;
                            const float nm = fmaxf(mx, sd), corr = __expf(mx - nm), e2 = __expf(sd - nm);
                            sum = sum * corr + e2;
#pragma unroll
                            for (int u = 0; u < 8; ++u) {
                                const int cidx = lane + 32 * u;
                                oacc[u] = oacc[u] * corr + (cidx < dh ? e2 * __ldcg(vj + cidx) : 0.f);
                            }
                            mx = nm;
                        }
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            const int cidx = lane + 32 * u;
                            if (cidx < dh)
                                ch_store_hi_lo(ph.att_out + (size_t)pos * p.d + (size_t)hd * dh + cidx, (size_t)p.lo_x * p.d, oacc[u] / sum);
                        }
                    }
                }
            }
            // this CTA's part of the phase is in memory: arrive at the grid barrier
            ch_epi_sync();
            if (t == 0) {
                *reinterpret_cast<volatile int *>(aux + kChAuxParked) = i + 1;    // also when nothing was parked
                __threadfence();
                atomicAdd(p.grid_bar, 1u);
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

// Sets the kernel's shared-memory limit (once per device: the attribute is per device) and asks
// whether `grid` CTAs of it can be resident together, which the phase barriers need: on a
// context that may use only part of the SMs (MPS with a thread percentage, a partitioned
// device) they cannot, and the caller then runs the chain as one kernel per GEMM.
template <int RP, int KC, bool MOD = false>
cudaError_t chain_prepare(int grid, size_t smem, int sm_count, bool *fits)
{
    auto kern = sk_chain_kernel<RP, KC, MOD>;
    static std::atomic<unsigned long long> attr_devices{0}, fit_devices{0}, nofit_devices{0};
    int dev = 0;
    cudaError_t ea = cudaGetDevice(&dev);
    if (ea != cudaSuccess) return ea;
    const unsigned long long bit = 1ull << (dev & 63);
    if (!(attr_devices.load() & bit)) {
        ea = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
        if (ea != cudaSuccess) return ea;
        attr_devices.fetch_or(bit);
    }
    if (!((fit_devices.load() | nofit_devices.load()) & bit)) {
        int per_sm = 0;
        ea = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kChThreads, smem);
        if (ea != cudaSuccess) return ea;
        ((long long)per_sm * sm_count >= grid ? fit_devices : nofit_devices).fetch_or(bit);
    }
    if (fits) *fits = (fit_devices.load() & bit) != 0;
    return cudaSuccess;
}

template <int RP, int KC, bool MOD = false>
cudaError_t chain_launch(const typename ChainTypes<MOD>::Maps &maps, const typename ChainTypes<MOD>::Params &p, int grid,
                         size_t smem, cudaStream_t st)
{
    auto kern = sk_chain_kernel<RP, KC, MOD>;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kChThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    // the CTAs wait for one another at the phase barriers: they must all be resident
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeCooperative;
    at[0].val.cooperative = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, maps, p);
}

}  // namespace

// The whole head chain (K heads) for M <= 128 rows as one kernel.  Returns cudaErrorNotSupported
// (nothing launched) if the shape does not fit this form; the caller then runs the chain as
// separate kernels.
cudaError_t sk_chain(Ctx *c, int M, int K, const mrp_draft_out &out, cudaStream_t st, bool f16_lm, bool check_only)
{
    const TcState *s = (const TcState *)c->tc_state;
    const int d = c->cfg.d, F = c->cfg.d_ff, G = c->sm_count;
    if (K < 1 || K > 4 || 2 * K > kChMaxPhases || M < 1 || M > 128) return cudaErrorNotSupported;
    // Measured against one kernel per GEMM (programmatic dependent launch between them), whole
    // mrp_draft call: d = 2048, F = 4096, M = 4, K = 3: 60 vs 77 us for the heads; d = 4096,
    // F = 8192: M = 1, K = 1 0.244 vs 0.247 ms, M = 4, K = 4 0.371 vs 0.378 ms, M = 16, K = 4
    // 0.398 vs 0.412 ms, M = 64, K = 1 69 vs 84 us for the head (M = 16, K = 1 is the one point
    // where the separate kernels are ahead, by 2 us).  So every shape that fits runs here.
    const int r_pad = sk_head_pad(M);
    const int gu_tiles = F / 64, dn_tiles = (d + 127) / 128;
    if (gu_tiles > G || dn_tiles > G || G > kSumsqSlices || gu_tiles > kChTilesPerPhase ||
        kChMaxPhases * kChTilesPerPhase >= kSkMaxTiles)
        return cudaErrorNotSupported;
    if ((size_t)G * r_pad * 128 * 4 > (size_t)kSkScratchBytes) return cudaErrorNotSupported;

    {
        // a down-projection share must fit the shared-memory buffer of squares
        int S = G / dn_tiles;
        if (S < 1) S = 1;
        if (S > F / kBK) S = F / kBK;
        const int cps = (F / kBK + S - 1) / S;
        S = (F / kBK + cps - 1) / cps;
        if (M * ((128 + S - 1) / S) > kChMaxShare) return cudaErrorNotSupported;
    }
    auto split = [&](int n_tiles, int k_chunks) {
        int S = G / n_tiles;
        if (S < 1) S = 1;
        if (S > k_chunks) S = k_chunks;
        const int cps = (k_chunks + S - 1) / S;
        return (k_chunks + cps - 1) / cps;          // no empty slice
    };
    const int gu_split = split(gu_tiles, d / kBK), dn_split = split(dn_tiles, F / kBK);
    // two k-chunks per ring stage where every slice of both GEMMs has an even number of them
    const bool even = (d / kBK) % (2 * gu_split) == 0 && (F / kBK) % (2 * dn_split) == 0;
    const int kc = (even && r_pad <= 32) ? 2 : 1;
    const int stage = kc * (kChWTile + 2 * r_pad * 128);
    int ns = (kSmemBudget - 1024 - 256 - 16 - kChAuxBytes) / stage;
    if (ns > 12) ns = 12;
    const size_t smem = (size_t)ns * stage + 1024 + 8 * (2 * ns + 4) + 16 + kChAuxBytes;
    {
        // all G CTAs must be resident at once (they wait for one another)
        bool fits = false;
        cudaError_t eq;
        switch (r_pad) {
        case 16: eq = kc == 2 ? chain_prepare<16, 2>(G, smem, G, &fits) : chain_prepare<16, 1>(G, smem, G, &fits); break;
        case 32: eq = kc == 2 ? chain_prepare<32, 2>(G, smem, G, &fits) : chain_prepare<32, 1>(G, smem, G, &fits); break;
        case 64: eq = chain_prepare<64, 1>(G, smem, G, &fits); break;
        default: eq = chain_prepare<128, 1>(G, smem, G, &fits); break;
        }
        if (eq != cudaSuccess || !fits) return cudaErrorNotSupported;
    }
    if (check_only) return cudaSuccess;

    ChainParams p;
    memset(&p, 0, sizeof(p));
    ChainMaps maps;
    memset(&maps, 0, sizeof(maps));
    const int n_rs = (K + 1) * M;
    p.n_phases = 2 * K; p.M = M; p.d = d; p.F = F; p.n_rs = n_rs; p.eps = c->cfg.rms_eps;
    p.lo_x = c->lo_x; p.lo_xt = c->lo_xt;
    p.act = (__nv_bfloat16 *)(c->ws + c->lay.act);
    p.hcur = (float *)(c->ws + c->lay.hcur); p.h0f = (const float *)(c->ws + c->lay.h0f);
    p.ssq_fix = (unsigned long long *)(c->ws + c->lay.ssq_fix);
    p.scratch = (float *)(c->ws + c->lay.sk_scratch);
    p.counters = (int32_t *)(c->ws + c->lay.sk_counters);
    p.grid_bar = (unsigned int *)(c->ws + c->lay.sk_counters) + (kSkMaxTiles - 1);
    p.status = (int32_t *)(c->ws + c->lay.status); p.user_status = out.status;
    p.n_stages = ns;
    int cols = 32;
    while (cols < 2 * 2 * r_pad) cols <<= 1;
    p.tmem_cols = cols;

    __nv_bfloat16 *xg = (__nv_bfloat16 *)(c->ws + c->lay.xg);
    __nv_bfloat16 *xt = (__nv_bfloat16 *)(c->ws + c->lay.xt);
    if (!make_map(s, &maps.m[0], xg, d, 2 * (uint64_t)r_pad, 2 * r_pad) ||
        !make_map(s, &maps.m[1], p.act, F, 2 * (uint64_t)r_pad, 2 * r_pad))
        return note_err(c, cudaErrorInvalidValue, "tensor map (head chain, activations)");
    for (int k = 1; k <= K; ++k) {
        const mrp_head_weights &hw = c->heads[k - 1];
        const int b = 2 + 3 * (k - 1);
        if (!make_map(s, &maps.m[b], hw.w_gate, d, F, 64) || !make_map(s, &maps.m[b + 1], hw.w_up, d, F, 64) ||
            !make_map(s, &maps.m[b + 2], hw.w_down, F, d, 128))
            return note_err(c, cudaErrorInvalidValue, "tensor map (head chain, weights)");
        ChainPhase &gu = p.ph[2 * (k - 1)], &dn = p.ph[2 * (k - 1) + 1];
        gu.kind = CH_GU; gu.k_chunks = d / kBK; gu.n_tiles = gu_tiles; gu.n_split = gu_split;
        gu.w_rows = F; gu.map_x = 0; gu.map_w0 = b; gu.map_w1 = b + 1;
        gu.ssq_idx = k - 1;
        dn.kind = CH_DN; dn.k_chunks = F / kBK; dn.n_tiles = dn_tiles; dn.n_split = dn_split;
        if (M * ((128 + dn.n_split - 1) / dn.n_split) > kChMaxShare) return cudaErrorNotSupported;
        dn.ssq_idx = k;
        dn.w_rows = d; dn.map_x = 1; dn.map_w0 = b + 2; dn.map_w1 = b + 2;
        dn.gamma_next = (k < K) ? (const __nv_bfloat16 *)c->heads[k].rms_gamma : nullptr;
        dn.xg_next = (k < K) ? xg : nullptr;
        dn.xt_k = xt + (size_t)k * M * d;
        dn.xt16_k = f16_lm ? (__half *)(c->ws + c->lay.xt16) + (size_t)(k - (c->from_hidden ? 0 : 1)) * M * d : nullptr;
        dn.hidden_out = (k == K) ? out.hidden_out : nullptr;
    }
    cudaError_t e;
    switch (r_pad) {
    case 16: e = kc == 2 ? chain_launch<16, 2>(maps, p, G, smem, st) : chain_launch<16, 1>(maps, p, G, smem, st); break;
    case 32: e = kc == 2 ? chain_launch<32, 2>(maps, p, G, smem, st) : chain_launch<32, 1>(maps, p, G, smem, st); break;
    case 64: e = chain_launch<64, 1>(maps, p, G, smem, st); break;
    default: e = chain_launch<128, 1>(maps, p, G, smem, st); break;
    }
    c->launches++;
    return note_err(c, e, "head-chain kernel");
}

// One step of the token-conditioned module (Sec. 3.2) over n <= 128 positions as ONE cooperative kernel: the rows
// [h ; emb[x]] -> fusion projection -> per layer q/k/v (three matrices, one product) -> attention -> output projection
// -> gate/up -> down projection -> h <- h + Delta and the LM-head operand of the masked rows, as phases of the
// head-chain kernel's machinery (split contraction, slices finished by all CTAs, weights of the next phase prefetched
// before the grid barrier).  Operands in the few-row form (lo rows sk_head_pad(n) rows behind the hi rows); the sums
// of squares of the norms live in slots of the fixed-point array.  `bar_mem`: kModChainPhases * kChTilesPerPhase + 1
// zero-able counters of the caller's (module workspace).  cudaErrorNotSupported (nothing launched): the shape does
// not fit; the caller runs the products as separate kernels.
cudaError_t sk_module_step(Ctx *c, int n, int L, const int32_t *tokens, const void *hidden0, float *h_state, bool first_step,
                           __nv_bfloat16 *cat16, __nv_bfloat16 *xa, __nv_bfloat16 *xb, __nv_bfloat16 *act16, float *q, float *k,
                           float *v, float *z, int32_t *bar_mem, const int32_t *row_index, int n_masked, int lo_xt, bool f16_lm,
                           float *hidden_out, int32_t *user_status, cudaStream_t st, bool check_only, float *att_part,
                           int *att_counters)
{
    const TcState *s = (const TcState *)c->tc_state;
    const mrp_module_weights &w = c->module;
    const int d = c->cfg.d, F = c->cfg.d_ff, G = c->sm_count, D = w.n_layers, H = w.n_attn_heads;
    if (D < 1 || D > kModChainLayers || n < 1 || n > 128 || d % 128 || F % 64 || d / H > 256 || (d / H) % 32)
        return cudaErrorNotSupported;
    // (the clean-prefix attention stages a tile of queries and the four warps' partial results in the 16 KB of
    // shared memory the phases share)
    if (c->has_prefix && att_sh_floats(d / H) > 4096) return cudaErrorNotSupported;
    const int r_pad = sk_head_pad(n);
    const int d_tiles = d / 128, gu_tiles = F / 64;
    if (3 * d_tiles > G || gu_tiles > G || 3 * d_tiles > kChTilesPerPhase || gu_tiles > kChTilesPerPhase ||
        (size_t)G * r_pad * 128 * 4 > (size_t)kSkScratchBytes)
        return cudaErrorNotSupported;
    auto split = [&](int n_tiles, int k_chunks) {
        int S = G / n_tiles;
        if (S < 1) S = 1;
        if (S > k_chunks) S = k_chunks;
        const int cps = (k_chunks + S - 1) / S;
        return (k_chunks + cps - 1) / cps;          // no empty slice
    };
    const int sp_proj = split(d_tiles, 2 * d / kBK), sp_qkv = split(3 * d_tiles, d / kBK), sp_o = split(d_tiles, d / kBK);
    const int sp_gu = split(gu_tiles, d / kBK), sp_dn = split(d_tiles, F / kBK);
    // (the products with a norm behind them keep a share's squares in shared memory)
    auto share_fits = [&](int sp) { return n * ((128 + sp - 1) / sp) <= kChMaxShare; };
    if (!share_fits(sp_o) || !share_fits(sp_dn) || !share_fits(sp_proj)) return cudaErrorNotSupported;
    const int stage = kChWTile + 2 * r_pad * 128;           // one k-chunk per ring stage
    int ns = (kSmemBudget - 1024 - 256 - 16 - kChAuxBytes) / stage;
    if (ns > 12) ns = 12;
    const size_t smem = (size_t)ns * stage + 1024 + 8 * (2 * ns + 4) + 16 + kChAuxBytes;
    {
        bool fits = false;
        cudaError_t eq;
        switch (r_pad) {
        case 16: eq = chain_prepare<16, 1, true>(G, smem, G, &fits); break;
        case 32: eq = chain_prepare<32, 1, true>(G, smem, G, &fits); break;
        case 64: eq = chain_prepare<64, 1, true>(G, smem, G, &fits); break;
        default: eq = chain_prepare<128, 1, true>(G, smem, G, &fits); break;
        }
        if (eq != cudaSuccess || !fits) return cudaErrorNotSupported;
    }
    if (check_only) return cudaSuccess;

    ModChainParams p;
    memset(&p, 0, sizeof(p));
    ModChainMaps maps;
    memset(&maps, 0, sizeof(maps));
    p.M = n; p.d = d; p.F = F; p.eps = c->cfg.rms_eps; p.lo_x = r_pad; p.lo_xt = lo_xt;
    p.act = act16;
    p.ssq_fix = (unsigned long long *)(c->ws + c->lay.ssq_fix);
    p.scratch = (float *)(c->ws + c->lay.sk_scratch);
    p.counters = bar_mem;
    p.grid_bar = (unsigned int *)bar_mem + kModChainPhases * kChTilesPerPhase;
    p.status = (int32_t *)(c->ws + c->lay.status); p.user_status = user_status;
    p.n_stages = ns;
    int cols = 32;
    while (cols < 2 * 2 * r_pad) cols <<= 1;
    p.tmem_cols = cols;
    p.mod.tokens = tokens; p.mod.hidden0 = (const __nv_bfloat16 *)hidden0; p.mod.emb = (const __nv_bfloat16 *)w.emb;
    p.mod.h_state = h_state; p.mod.z = z; p.mod.cat = cat16; p.mod.first_step = first_step ? 1 : 0;
    p.mod.mask_token = w.mask_token; p.mod.emb_rows = w.emb_rows; p.mod.row_index = row_index; p.mod.n_masked = n_masked;
    p.mod.xt = (__nv_bfloat16 *)(c->ws + c->lay.xt); p.mod.xt16 = f16_lm ? (__half *)(c->ws + c->lay.xt16) : nullptr;
    p.mod.hidden_out = hidden_out;
    if (c->has_prefix) {
        const void *ptrs[2 * kModChainLayers];
        for (int l = 0; l < D; ++l) { ptrs[2 * l] = c->prefix_layers[l].k; ptrs[2 * l + 1] = c->prefix_layers[l].v; }
        const bool mma = att_mma_ok(c->prefix_cap, L, (n / L) * H, d, d / H, ptrs, 2 * D);
        const AttSplit sp = mma ? att_split_mma(c->prefix_cap, L, (n / L) * H, d / H, G) : att_split(c->prefix_cap, L, (n / L) * H, d / H, G);
        p.mod.plen = c->prefix_len; p.mod.pcap = c->prefix_cap; p.mod.append = c->prefix_append ? 1 : 0;
        p.mod.att_nch = sp.n_ch; p.mod.att_gpc = sp.gpc; p.mod.att_mma = mma ? 1 : 0;
        p.mod.att_part = att_part; p.mod.att_counters = att_counters;
    }
    bool ok = make_map(s, &maps.m[0], xa, d, 2 * (uint64_t)r_pad, 2 * r_pad) && make_map(s, &maps.m[1], act16, F, 2 * (uint64_t)r_pad, 2 * r_pad) &&
              make_map(s, &maps.m[2], xb, d, 2 * (uint64_t)r_pad, 2 * r_pad) &&
              make_map(s, &maps.m[3], cat16, 2 * d, 2 * (uint64_t)r_pad, 2 * r_pad) && make_map(s, &maps.m[4], w.w_proj, 2 * d, d, 128);
    for (int l = 0; l < D && ok; ++l) {
        const mrp_module_layer &y = w.layers[l];
        const int b = 5 + 7 * l;
        ok = make_map(s, &maps.m[b], y.w_q, d, d, 128) && make_map(s, &maps.m[b + 1], y.w_k, d, d, 128) &&
             make_map(s, &maps.m[b + 2], y.w_v, d, d, 128) && make_map(s, &maps.m[b + 3], y.w_o, d, d, 128) &&
             make_map(s, &maps.m[b + 4], y.w_gate, d, F, 64) && make_map(s, &maps.m[b + 5], y.w_up, d, F, 64) &&
             make_map(s, &maps.m[b + 6], y.w_down, F, d, 128);
    }
    if (!ok) return note_err(c, cudaErrorInvalidValue, "tensor map (module step)");
    int i = 0;
    auto plain = [&](int kind) -> ChainPhase & {           // a phase without a product
        ChainPhase &ph = p.ph[i++];
        ph.kind = kind; ph.n_tiles = 0; ph.n_split = 1; ph.k_chunks = 1; ph.ssq_in = -1; ph.zero_slot0 = -1; ph.zero_slot1 = -1;
        return ph;
    };
    auto lin = [&](int k_chunks, int n_tiles, int n_split, int map_x, int map_w) -> ChainPhase & {
        ChainPhase &ph = p.ph[i++];
        ph.kind = CH_LIN; ph.k_chunks = k_chunks; ph.n_tiles = n_tiles; ph.n_split = n_split; ph.w_rows = d;
        ph.map_x = map_x; ph.map_w0 = map_w; ph.map_w1 = map_w; ph.ssq_in = -1; ph.zero_slot0 = -1; ph.zero_slot1 = -1;
        return ph;
    };
    // slots of the fixed-point sums of squares: 0 / 1 alternate as the attention norm of layer l / l + 1, 3 is the MLP norm;
    // slot 0 is cleared before the launch, the others by the first phase
    const int s_mlp = 3;
    {
        ChainPhase &ph = plain(CH_CAT);
        ph.zero_slot0 = 1; ph.zero_slot1 = s_mlp;
    }
    {
        ChainPhase &ph = lin(2 * d / kBK, d_tiles, sp_proj, 3, 4);
        ph.lin_out = z; ph.gamma_next = (const __nv_bfloat16 *)w.layers[0].g_attn; ph.xg_next = xa; ph.ssq_idx = 0;
    }
    for (int l = 0; l < D; ++l) {
        const mrp_module_layer &y = w.layers[l];
        const int b = 5 + 7 * l, s_in = l & 1, s_next = 1 - s_in;
        {
            ChainPhase &ph = lin(d / kBK, 3 * d_tiles, sp_qkv, 0, b);
            ph.lin_out = q; ph.lin_out1 = k; ph.lin_out2 = v; ph.lin3_tiles = d_tiles; ph.ssq_in = s_in;
            if (l > 0) { ph.zero_slot0 = s_next; ph.zero_slot1 = s_mlp; }     // (their readers are behind us, their writers ahead)
        }
        {
            ChainPhase &ph = plain(CH_ATT);
            ph.att_q = q; ph.att_k = k; ph.att_v = v; ph.att_out = xb; ph.att_L = L; ph.att_H = H;
            if (c->has_prefix) {
                ph.att_pk = (__nv_bfloat16 *)c->prefix_layers[l].k;
                ph.att_pv = (__nv_bfloat16 *)c->prefix_layers[l].v;
            }
        }
        {
            ChainPhase &ph = lin(d / kBK, d_tiles, sp_o, 2, b + 3);
            ph.lin_out = z; ph.lin_acc = 1; ph.gamma_next = (const __nv_bfloat16 *)y.g_mlp; ph.xg_next = xa; ph.ssq_idx = s_mlp;
        }
        {
            ChainPhase &ph = p.ph[i++];
            ph.kind = CH_GU; ph.k_chunks = d / kBK; ph.n_tiles = gu_tiles; ph.n_split = sp_gu; ph.w_rows = F;
            ph.map_x = 0; ph.map_w0 = b + 4; ph.map_w1 = b + 5; ph.ssq_idx = s_mlp; ph.ssq_in = -1; ph.zero_slot0 = -1; ph.zero_slot1 = -1;
        }
        {
            ChainPhase &ph = lin(F / kBK, d_tiles, sp_dn, 1, b + 6);
            const void *g_next = l + 1 < D ? w.layers[l + 1].g_attn : nullptr;
            ph.lin_out = z; ph.lin_acc = 1;
            ph.gamma_next = (const __nv_bfloat16 *)g_next; ph.xg_next = g_next ? xa : nullptr; ph.ssq_idx = s_next;
            ph.fin = l + 1 == D ? 1 : 0;       // Delta complete: h <- h + Delta and the LM-head operand in the same finish
        }
    }
    p.n_phases = i;
    // arrival counters, the grid barrier and the first slot of the sums of squares start at zero
    cudaError_t e = cudaMemsetAsync(bar_mem, 0, ((size_t)kModChainPhases * kChTilesPerPhase + 1) * 4, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(c->ws + c->lay.ssq_fix, 0, (size_t)128 * 8, st);
    if (e != cudaSuccess) return note_err(c, e, "module step, counters");
    switch (r_pad) {
    case 16: e = chain_launch<16, 1, true>(maps, p, G, smem, st); break;
    case 32: e = chain_launch<32, 1, true>(maps, p, G, smem, st); break;
    case 64: e = chain_launch<64, 1, true>(maps, p, G, smem, st); break;
    default: e = chain_launch<128, 1, true>(maps, p, G, smem, st); break;
    }
    c->launches++;
    return note_err(c, e, "module step kernel");
}

}  // namespace mrp
