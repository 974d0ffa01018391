// Reveal selection, remasking and draft verification: one warp per (sequence, block).
//
// STATIC   (Algorithm 2, reveal step at k = 0..K; Algorithm 3, draft step after each MRP
//           update): for k = 0..K the r most confident still-masked
//           positions under step k, confidence descending then position ascending.
// DYNAMIC  (Algorithm 4; Sec. 4.1 dynamic denoising; Sec. 4.4 cap): R = {conf_0 >= tau},
//           at least one, optionally capped; remask members of R whose updated confidence
//           is below the same tau.
// VERIFY   (Algorithm 3, rejection step: a draft that differs from the backbone's argmax is
//           rejected; Figure 1(d): prefix acceptance).
// Lane l owns block positions l, l+32, ... (up to 32 strides, i.e. L <= 1024); membership
// sets are per-lane bit masks over the strides.
#include <limits.h>

#include <mutex>

#include "mrp_internal.cuh"

namespace mrp {

__device__ __forceinline__ void raise_bad_index(int32_t *status, int32_t *user_status)
{
    if (status) atomicOr(status, MRP_DEV_BAD_INDEX);
    if (user_status) atomicOr(user_status, MRP_DEV_BAD_INDEX);
}

// dense_row[position] = masked row, over n_pos = B * L positions preset to -1.  A row whose
// position is outside [0, n_pos) is skipped; of several rows naming one position the one listed
// last (highest m) keeps it, whatever the order the threads run in.  Both raise MRP_DEV_BAD_INDEX.
__global__ void scatter_rows_kernel(const int32_t *__restrict__ row_index, int M, int n_pos,
                                    int32_t *__restrict__ dense_row, int32_t *__restrict__ status,
                                    int32_t *__restrict__ user_status)
{
    const int m = blockIdx.x * blockDim.x + threadIdx.x;
    if (m >= M) return;
    const int idx = row_index ? row_index[m] : m;
    if (!row_ok(idx, n_pos)) { raise_bad_index(status, user_status); return; }
    if (atomicMax(dense_row + idx, m) != -1) raise_bad_index(status, user_status);
}

// Most confident position among the lanes' candidate bit sets under confidences c[row]:
// (confidence desc, position asc).  Returns the block position or INT_MAX if none.
__device__ __forceinline__ int warp_best(uint32_t cand, const float *__restrict__ c,
                                         const int32_t *__restrict__ rows, int lane)
{
    float bc = -INFINITY;
    int bi = INT_MAX;
    while (cand) {
        const int s = __ffs(cand) - 1;
        cand &= cand - 1;
        const int i = lane + 32 * s;
        const float v = c[rows[i]];
        if (bi == INT_MAX || v > bc || (v == bc && i < bi)) { bc = v; bi = i; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float oc = __shfl_xor_sync(0xffffffffu, bc, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (oi != INT_MAX && (bi == INT_MAX || oc > bc || (oc == bc && oi < bi))) { bc = oc; bi = oi; }
    }
    return bi;
}

__device__ __forceinline__ int warp_popc(uint32_t bits)
{
    int n = __popc(bits);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) n += __shfl_xor_sync(0xffffffffu, n, o);
    return n;
}

__global__ void __launch_bounds__(32)
select_kernel(const float *__restrict__ conf, const int32_t *__restrict__ token,
              const int32_t *__restrict__ dense_row, int M, int K, int L, mrp_select_params p,
              mrp_select_out out, int Kd, const int32_t *__restrict__ row_index, int32_t *__restrict__ status)
{
    pdl_trigger();
    pdl_wait();
    const int b = blockIdx.x, lane = threadIdx.x;
    // Position -> masked row of this block: from the prepared dense map, or (dense_row == NULL,
    // few masked rows) built here in shared memory by one scan over the row list.
    __shared__ int32_t rows_s[1024];
    const int32_t *rows = rows_s;
    if (dense_row) {
        rows = dense_row + (size_t)b * L;
    } else {
        for (int i = lane; i < L; i += 32) rows_s[i] = -1;
        __syncwarp();
        // rows of other blocks are skipped, and with them any index outside [0, B * L) (block 0
        // reports those); of several rows naming one position the one listed last keeps it
        const long long lo = (long long)b * L, n_pos = (long long)gridDim.x * L;
        for (int m = lane; m < M; m += 32) {
            const long long idx = row_index ? row_index[m] : m;
            if (idx >= lo && idx < lo + L) {
                if (atomicMax(&rows_s[idx - lo], m) != -1) raise_bad_index(status, out.status);
            } else if (b == 0 && (idx < 0 || idx >= n_pos)) {
                raise_bad_index(status, out.status);
            }
        }
        __syncwarp();
    }
    int8_t *reveal = out.reveal_mask + (size_t)b * L, *remask = out.remask_mask + (size_t)b * L;
    int32_t *otok = out.out_token + (size_t)b * L;
    int8_t *step = out.step_of + (size_t)b * L;
    for (int i = lane; i < L; i += 32) { reveal[i] = 0; remask[i] = 0; otok[i] = -1; step[i] = -1; }
    for (int q = lane; q < Kd; q += 32) {
        out.draft_pos[(size_t)b * Kd + q] = -1;
        out.draft_tok[(size_t)b * Kd + q] = -1;
    }
    __syncwarp();
    uint32_t avail = 0;
    for (int s = 0; lane + 32 * s < L; ++s)
        if (rows[lane + 32 * s] >= 0) avail |= 1u << s;
    const int n = warp_popc(avail);
    int dl = 0;
    if (n > 0 && p.mode == MRP_SELECT_STATIC) {
        for (int k = 0; k <= K; ++k) {
            const int r = (k == 0) ? p.r_reveal : p.r_draft;
            const float *ck = conf + (size_t)k * M;
            for (int t = 0; t < r; ++t) {
                const int bi = warp_best(avail, ck, rows, lane);
                if (bi == INT_MAX) break;
                if ((bi & 31) == lane) {
                    avail &= ~(1u << (bi >> 5));
                    const int32_t tk = token[(size_t)k * M + rows[bi]];
                    otok[bi] = tk;
                    step[bi] = (int8_t)k;
                    if (k == 0) {
                        reveal[bi] = 1;
                    } else {
                        out.draft_pos[(size_t)b * Kd + dl] = bi;
                        out.draft_tok[(size_t)b * Kd + dl] = tk;
                    }
                }
                if (k > 0) ++dl;
            }
        }
    } else if (n > 0) {
        uint32_t inR = 0;
        for (uint32_t c = avail; c; c &= c - 1) {
            const int s = __ffs(c) - 1;
            if (conf[rows[lane + 32 * s]] >= p.tau) inR |= 1u << s;
        }
        int nR = warp_popc(inR);
        if (nR == 0 && p.ensure_progress) {
            const int bi = warp_best(avail, conf, rows, lane);
            if ((bi & 31) == lane) inR |= 1u << (bi >> 5);
            nR = 1;
        }
        if (p.use_cap) {
            int cap = (7 * n) / 10;
            cap = cap < 5 ? 5 : cap;
            cap = cap > L ? L : cap;
            if (nR > cap) {
                uint32_t cand = inR, keep = 0;
                for (int t = 0; t < cap; ++t) {
                    const int bi = warp_best(cand, conf, rows, lane);
                    if ((bi & 31) == lane) { cand &= ~(1u << (bi >> 5)); keep |= 1u << (bi >> 5); }
                }
                inR = keep;
                nR = cap;
            }
        }
        uint32_t rem = 0;
        for (uint32_t c = inR; c; c &= c - 1) {
            const int s = __ffs(c) - 1;
            const int m = rows[lane + 32 * s];
            bool revoke;
            if (p.remask_policy == 3) {
                // the argmax moved away from the revealed token at some step
                revoke = false;
                for (int k = 1; k <= K; ++k) revoke |= token[(size_t)k * M + m] != token[m];
            } else {
                // policy 2 follows the revealed token's own probability instead of the top one
                const float *cu = (p.remask_policy == 2) ? p.conf_first : conf;
                float c2;
                if (K == 0) {
                    c2 = cu[m];
                } else if (p.remask_policy == 1) {
                    c2 = cu[(size_t)K * M + m];
                } else {
                    c2 = cu[(size_t)M + m];
                    for (int k = 2; k <= K; ++k) c2 = fminf(c2, cu[(size_t)k * M + m]);
                }
                revoke = c2 < p.tau;
            }
            if (revoke) rem |= 1u << s;
        }
        const int kept = warp_popc(inR & ~rem);
        if (kept == 0 && nR > 0 && p.ensure_progress) {
            const int bi = warp_best(inR, conf, rows, lane);
            if ((bi & 31) == lane) rem &= ~(1u << (bi >> 5));
        }
        for (uint32_t c = inR; c; c &= c - 1) {
            const int s = __ffs(c) - 1;
            const int i = lane + 32 * s;
            reveal[i] = 1;
            if (rem & (1u << s)) {
                remask[i] = 1;
            } else {
                otok[i] = token[rows[i]];
                step[i] = 0;
            }
        }
    }
    if (lane == 0) out.draft_len[b] = dl;
}

__global__ void verify_kernel(const int32_t *__restrict__ draft_tok,
                              const int32_t *__restrict__ verify_tok,
                              const int32_t *__restrict__ draft_len, int B, int Kd, int positionwise,
                              int32_t *__restrict__ accept_len, int8_t *__restrict__ accept_mask)
{
    pdl_trigger();
    pdl_wait();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    int n = draft_len[b];
    n = n > Kd ? Kd : (n < 0 ? 0 : n);
    int acc = 0;
    bool alive = true;
    for (int j = 0; j < Kd; ++j) {
        bool ok = (j < n) && (draft_tok[(size_t)b * Kd + j] == verify_tok[(size_t)b * Kd + j]);
        if (!positionwise) { alive = alive && ok; ok = alive; }
        accept_mask[(size_t)b * Kd + j] = (int8_t)ok;
        acc += ok;
    }
    accept_len[b] = acc;
}

cudaError_t launch_select(Ctx *c, const float *conf, const int32_t *token, const int32_t *row_index,
                          int M, int K, int B, int L, const mrp_select_params &p,
                          const mrp_select_out &out, cudaStream_t st)
{
    const int Kd = K * (p.r_draft > 0 ? p.r_draft : 0);
    int32_t *status = (int32_t *)(c->ws + c->lay.status);
    if ((long long)B * M <= (1ll << 22)) {
        // few rows: every block finds its rows itself, one launch instead of three
        c->launches++;
        return launch_k(select_kernel, dim3(B), dim3(32), 0, st, !(c->cfg.flags & MRP_FLAG_NO_PDL), conf, token,
                        (const int32_t *)nullptr, M, K, L, p, out, Kd, row_index, status);
    }
    int32_t *dense_row = (int32_t *)(c->ws + c->lay.dense_row);
    cudaError_t e = cudaMemsetAsync(dense_row, 0xFF, sizeof(int32_t) * (size_t)B * L, st);
    if (e != cudaSuccess) return e;
    if (M > 0) {
        scatter_rows_kernel<<<(M + 255) / 256, 256, 0, st>>>(row_index, M, B * L, dense_row, status, out.status);
        c->launches++;
    }
    select_kernel<<<B, 32, 0, st>>>(conf, token, dense_row, M, K, L, p, out, Kd, nullptr, status);
    c->launches++;
    return cudaGetLastError();
}

cudaError_t launch_verify(Ctx *c, const int32_t *draft_tok, const int32_t *verify_tok,
                          const int32_t *draft_len, int B, int Kd, int positionwise,
                          int32_t *accept_len, int8_t *accept_mask, cudaStream_t st)
{
    if (B == 0) return cudaSuccess;
    c->launches++;
    return launch_k(verify_kernel, dim3((B + 127) / 128), dim3(128), 0, st, !(c->cfg.flags & MRP_FLAG_NO_PDL),
                    draft_tok, verify_tok, draft_len, B, Kd, positionwise, accept_len, accept_mask);
}

// ---- block-state transition x_t -> x_{t-1}: one warp per block -----------------------------
__global__ void commit_kernel(int32_t *__restrict__ tokens, const int32_t *__restrict__ out_token,
                              const int8_t *__restrict__ step_of, const int32_t *__restrict__ draft_pos,
                              const int32_t *__restrict__ draft_tok, const int8_t *__restrict__ accept_mask,
                              int L, int Kd, int32_t *__restrict__ block_masked)
{
    pdl_trigger();
    pdl_wait();
    const int b = blockIdx.x, lane = threadIdx.x;
    int32_t *tk = tokens + (size_t)b * L;
    for (int i = lane; i < L; i += 32) {
        const size_t p = (size_t)b * L + i;
        if (tk[i] >= 0) continue;
        const int32_t t = out_token[p];
        if (accept_mask ? (step_of[p] == 0) : (t >= 0)) tk[i] = t;
    }
    __syncwarp();
    if (accept_mask) {
        // accepted drafts (distinct positions of this block)
        for (int s = lane; s < Kd; s += 32) {
            const int pos = draft_pos[(size_t)b * Kd + s];
            if (accept_mask[(size_t)b * Kd + s] && pos >= 0 && pos < L && tk[pos] < 0) tk[pos] = draft_tok[(size_t)b * Kd + s];
        }
        __syncwarp();
    }
    int n = 0;
    for (int i0 = 0; i0 < L; i0 += 32) {
        const int i = i0 + lane;
        n += __popc(__ballot_sync(0xffffffffu, i < L && tk[i] < 0));
    }
    if (lane == 0) block_masked[b] = n;
}

// Exclusive prefix sum of the per-block counts (one CTA; counts of 1024 blocks per round).
__global__ void __launch_bounds__(1024) commit_scan_kernel(const int32_t *__restrict__ block_masked, int B,
                                                           int32_t *__restrict__ block_off, int32_t *__restrict__ n_masked)
{
    pdl_trigger();
    pdl_wait();
    __shared__ int warp_tot[32];
    __shared__ int carry_s;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) carry_s = 0;
    __syncthreads();
    for (int b0 = 0; b0 < B; b0 += 1024) {
        const int b = b0 + threadIdx.x;
        const int v = b < B ? block_masked[b] : 0;
        int inc = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += t;
        }
        if (lane == 31) warp_tot[warp] = inc;
        __syncthreads();
        int before = carry_s;
        for (int w = 0; w < warp; ++w) before += warp_tot[w];
        if (b < B) block_off[b] = before + inc - v;
        __syncthreads();
        if (threadIdx.x == 1023) carry_s = before + inc;
        __syncthreads();
    }
    if (threadIdx.x == 0) *n_masked = carry_s;
}

// Every block lists its still-masked positions, in order, from its offset on.
__global__ void commit_list_kernel(const int32_t *__restrict__ tokens, const int32_t *__restrict__ block_off, int L,
                                   int32_t *__restrict__ row_index)
{
    pdl_trigger();
    pdl_wait();
    const int b = blockIdx.x, lane = threadIdx.x;
    int off = block_off[b];
    for (int i0 = 0; i0 < L; i0 += 32) {
        const int i = i0 + lane;
        const bool masked = i < L && tokens[(size_t)b * L + i] < 0;
        const unsigned bal = __ballot_sync(0xffffffffu, masked);
        if (masked) row_index[off + __popc(bal & ((1u << lane) - 1u))] = b * L + i;
        off += __popc(bal);
    }
}

cudaError_t launch_commit(Ctx *c, const mrp_select_out &sel, const int8_t *accept_mask, int B, int L, int Kd,
                          const mrp_block_state &state, cudaStream_t st)
{
    const bool pdl = !(c->cfg.flags & MRP_FLAG_NO_PDL);
    int32_t *block_off = (int32_t *)(c->ws + c->lay.dense_row);     // B <= max_seqs entries fit
    cudaError_t e = launch_k(commit_kernel, dim3(B), dim3(32), 0, st, pdl, state.tokens, (const int32_t *)sel.out_token,
                             (const int8_t *)sel.step_of, (const int32_t *)sel.draft_pos, (const int32_t *)sel.draft_tok,
                             accept_mask, L, Kd, state.block_masked);
    if (e == cudaSuccess)
        e = launch_k(commit_scan_kernel, dim3(1), dim3(1024), 0, st, pdl, (const int32_t *)state.block_masked, B, block_off,
                     state.n_masked);
    if (e == cudaSuccess)
        e = launch_k(commit_list_kernel, dim3(B), dim3(32), 0, st, pdl, (const int32_t *)state.tokens,
                     (const int32_t *)block_off, L, state.row_index);
    c->launches += 3;
    return note_err(c, e, "commit kernels");
}

}  // namespace mrp

// ---------------------------------------------------------------------------------------
// Allocation-free selection entry point
// ---------------------------------------------------------------------------------------
// Some hosts of this library may not allocate device memory at all once they are running: a
// serving engine that handed the whole GPU to its own pool allocator, a plugin that lives
// inside someone else's CUDA context, code on a path where cudaMalloc would synchronise the
// device or is simply forbidden by policy.  Such a caller cannot provide the workspace a
// context needs, so reveal selection is offered once more with its only scratch (the dense
// position -> masked row map) in the fixed array below.  The array exists once per GPU that
// loads the library and is held until the process exits.
static __device__ __align__(256) int32_t mrp_noalloc_dense_row[MRP_NOALLOC_MAX_POSITIONS];

namespace {
// Device address of mrp_noalloc_dense_row, resolved on first use and remembered per (device,
// CUDA context): a module variable has one address per context, so a second context on the
// same device must not be handed the first one's pointer.  In host code the array's name is only
// a handle for the runtime, never a device address.
constexpr int kNoAllocSlots = 64;
struct NoAllocSlot { int dev; void *cuctx; int32_t *ptr; };
NoAllocSlot g_noalloc[kNoAllocSlots];
int g_noalloc_n = 0;
std::mutex g_noalloc_mu;

typedef int (*CtxGetCurrentFn)(void **);   // CUresult cuCtxGetCurrent(CUcontext *)

// The CUDA context current to this thread (nullptr if the driver entry point is not available:
// every call then resolves the address anew).
void *current_cuda_context()
{
    static CtxGetCurrentFn fn = nullptr;
    static bool looked = false;
    if (!looked) {
        void *f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuCtxGetCurrent", &f, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (CtxGetCurrentFn)f;
        looked = true;
    }
    void *cur = nullptr;
    if (!fn || fn(&cur) != 0) return nullptr;
    return cur;
}
}  // namespace

extern "C" int mrp_reveal_remask_noalloc(const float *conf, const int32_t *token,
                                         const int32_t *row_index, int32_t M, int32_t K, int32_t B,
                                         int32_t L, const mrp_select_params *params,
                                         const mrp_select_out *out, void *cuda_stream)
{
    using namespace mrp;
    if (!params || !out) return MRP_ERR_INVALID_ARG;
    if (B < 1 || L < 1 || L > 1024 || K < 0) return MRP_ERR_INVALID_ARG;
    if ((long long)B * L > (long long)MRP_NOALLOC_MAX_POSITIONS) return MRP_ERR_CAPACITY;
    if (M < 0 || (long long)M > (long long)B * L) return MRP_ERR_INVALID_ARG;
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

    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return MRP_ERR_CUDA;
    int32_t *dense_row = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_noalloc_mu);
        void *cuctx = current_cuda_context();      // nullptr before the thread has a context: resolve, do not remember
        for (int i = 0; i < g_noalloc_n && cuctx; ++i)
            if (g_noalloc[i].dev == dev && g_noalloc[i].cuctx == cuctx) dense_row = g_noalloc[i].ptr;
        if (!dense_row) {
            // once per (device, context), with that device current
            void *p = nullptr;
            if (cudaGetSymbolAddress(&p, mrp_noalloc_dense_row) != cudaSuccess || !p) return MRP_ERR_CUDA;
            dense_row = (int32_t *)p;
            if (cuctx && g_noalloc_n < kNoAllocSlots) g_noalloc[g_noalloc_n++] = NoAllocSlot{dev, cuctx, dense_row};
        }
    }
    cudaStream_t st = (cudaStream_t)cuda_stream;
    // the array still holds the previous call's map: every position of this call starts at -1
    if (cudaMemsetAsync(dense_row, 0xFF, sizeof(int32_t) * (size_t)B * L, st) != cudaSuccess)
        return MRP_ERR_CUDA;
    // rows whose position is outside [0, B * L) are skipped: nothing is written outside the part
    // of the array this call has just reset
    if (M > 0)
        scatter_rows_kernel<<<(M + 255) / 256, 256, 0, st>>>(row_index, M, B * L, dense_row, (int32_t *)nullptr,
                                                              out->status);
    select_kernel<<<B, 32, 0, st>>>(conf, token, dense_row, M, K, L, *params, *out, Kd, nullptr, (int32_t *)nullptr);
    return cudaGetLastError() == cudaSuccess ? MRP_OK : MRP_ERR_CUDA;
}
