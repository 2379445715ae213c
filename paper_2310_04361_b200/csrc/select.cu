// select_dynk (Eq. 4) and the routing metadata of Listing 1, all integer work after one
// float32 multiply per token, built from warp ballots, popcounts and prefix scans so that
// every output is unique and bit-exact: no sort, no order-dependent atomic.
//
//   mask kernel     one warp per token: row max, thr = tau*max (one fp32 RN multiply),
//                   ballot -> packed mask words, popcount -> k
//   count kernel    256 tokens per CTA; each warp turns its 32 tokens x 32 experts bit tile
//                   into per-expert token bitmaps with 32 ballots (a register transpose);
//                   the CTA that finishes last scans: per expert over the token blocks, then
//                   over the experts -> counts, offsets, n_sel
//   fill kernel     same tiling as the count kernel; rank of a token inside its expert's
//                   list = block base + popcounts of the warps before it + popcount of the
//                   lower lanes: tokens come out in ascending order
//   dual kernels    exclusive scan of k -> tok_off; one warp per token writes tok_exp
#include "d2d_common.cuh"

namespace {

constexpr int TOKB = 256;         // tokens per CTA in the count / fill kernels (8 warps x 32 tokens)
constexpr unsigned FULL = 0xffffffffu;

__device__ __forceinline__ bool is_finite_f32(float v) { return (__float_as_uint(v) & 0x7f800000u) != 0x7f800000u; }

// ---------------------------------------------------------------------------- mask kernels

// ksum (optional): [0] running sum of k over the CTAs, [1] exit ticket (both zero at launch and left at zero), [4]
// receives the total = number of selected (token, expert) pairs, for the density-adaptive dispatch of the expert step.
__global__ void __launch_bounds__(256)
dynk_mask_kernel(const float *__restrict__ R, int T, int E, int W, float tau,
                 uint32_t *__restrict__ mask, int32_t *__restrict__ k, int32_t *__restrict__ status, int32_t *ksum)
{
    __shared__ int block_k;
    if (ksum) {
        if (threadIdx.x == 0) block_k = 0;
        __syncthreads();
    }
    const int lane = threadIdx.x & 31;
    const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (t < T) {
        const float *row = R + (size_t)t * E;
        float m = -INFINITY;
        bool bad = false;
        for (int i = lane; i < E; i += 32) {
            const float v = __ldg(row + i);
            bad |= !is_finite_f32(v);
            m = v > m ? v : m;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float other = __shfl_xor_sync(FULL, m, o);
            m = other > m ? other : m;
        }
        bad = __any_sync(FULL, bad);
        const float thr = __fmul_rn(tau, m);     // the one rounding the rule is defined with
        int kt = 0;
        for (int w = 0; w < W; ++w) {
            const int i = w * 32 + lane;
            const bool keep = (i < E) && (bad || __ldg(row + i) >= thr);
            const uint32_t word = __ballot_sync(FULL, keep);
            if (lane == 0) mask[(size_t)t * W + w] = word;
            kt += __popc(word);
        }
        if (lane == 0) {
            k[t] = kt;
            if (bad) atomicMax(status, (int32_t)D2D_ERR_NONFINITE);
            if (ksum) atomicAdd(&block_k, kt);
        }
    }
    if (!ksum) return;
    __syncthreads();
    if (threadIdx.x == 0) {
        atomicAdd(ksum, block_k);
        __threadfence();
        if (atomicAdd(ksum + 1, 1) == (int)gridDim.x - 1) {          // the last CTA publishes the total and resets
            __threadfence();
            ksum[4] = atomicExch(ksum, 0);
            ksum[1] = 0;
        }
    }
}

// Static top-k: kk rounds of a warp arg-max over the not yet chosen experts; equal scores
// resolve to the lower expert index.  Lane l owns experts l, l+32, ... (bit j of `chosen`
// = expert l + 32 j), so the ballot of bit j over the lanes is exactly mask word j.
__global__ void __launch_bounds__(256)
topk_mask_kernel(const float *__restrict__ R, int T, int E, int W, int kk,
                 uint32_t *__restrict__ mask, int32_t *__restrict__ k, int32_t *__restrict__ status)
{
    const int lane = threadIdx.x & 31;
    const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (t >= T) return;
    const float *row = R + (size_t)t * E;
    bool bad = false;
    for (int i = lane; i < E; i += 32) bad |= !is_finite_f32(__ldg(row + i));
    bad = __any_sync(FULL, bad);
    unsigned long long chosen = 0ull;        // W <= 64 is checked on the host
    const int keep_n = bad ? E : min(kk, E);
    if (bad) {
        chosen = ~0ull;
    } else {
        for (int round = 0; round < keep_n; ++round) {
            float best = -INFINITY;
            int best_i = 0x7fffffff;
            for (int j = 0; j < W; ++j) {
                const int i = j * 32 + lane;
                if (i < E && !((chosen >> j) & 1ull)) {
                    const float v = __ldg(row + i);
                    if (v > best || (v == best && i < best_i)) { best = v; best_i = i; }
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float ov = __shfl_xor_sync(FULL, best, o);
                const int oi = __shfl_xor_sync(FULL, best_i, o);
                if (ov > best || (ov == best && oi < best_i)) { best = ov; best_i = oi; }
            }
            if ((best_i & 31) == lane && best_i < E) chosen |= 1ull << (best_i >> 5);
        }
    }
    for (int w = 0; w < W; ++w) {
        const bool keep = (w * 32 + lane < E) && ((chosen >> w) & 1ull);
        const uint32_t word = __ballot_sync(FULL, keep);
        if (lane == 0) mask[(size_t)t * W + w] = word;
    }
    if (lane == 0) {
        k[t] = keep_n;
        if (bad) atomicMax(status, (int32_t)D2D_ERR_NONFINITE);
    }
}

// k from a caller-supplied mask (override protocol of Sec. 4.4).
__global__ void __launch_bounds__(256)
k_from_mask_kernel(const uint32_t *__restrict__ mask, int T, int W, int32_t *__restrict__ k)
{
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= T) return;
    int kt = 0;
    for (int w = 0; w < W; ++w) kt += __popc(__ldg(mask + (size_t)t * W + w));
    k[t] = kt;
}

// ---------------------------------------------------------------------------- bucketing

// Lane j returns the bitmap, over this warp's 32 tokens, of bit j of `word`.
__device__ __forceinline__ uint32_t transpose_bits(uint32_t word, int lane)
{
    uint32_t col = 0;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        const uint32_t b = __ballot_sync(FULL, (word >> j) & 1u);
        if (lane == j) col = b;
    }
    return col;
}

// Exclusive scan of one int per thread over a 256-thread CTA; returns the exclusive prefix and
// leaves the CTA total in *total_out (shared).
__device__ __forceinline__ int block_exscan_256(int v, int *warp_sums /*[8]*/, int *total_out)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int n = __shfl_up_sync(FULL, inc, o);
        if (lane >= o) inc += n;
    }
    if (lane == 31) warp_sums[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        const int ws = lane < 8 ? warp_sums[lane] : 0;
        int winc = ws;
#pragma unroll
        for (int o = 1; o < 8; o <<= 1) {
            const int n = __shfl_up_sync(FULL, winc, o);
            if (lane >= o) winc += n;
        }
        if (lane < 8) warp_sums[lane] = winc - ws;
        if (lane == 7) *total_out = winc;
    }
    __syncthreads();
    const int res = warp_sums[warp] + inc - v;
    __syncthreads();
    return res;
}

// Per-expert token counts of each 256-token block (8 warps x 32 tokens; a warp turns its
// 32 x 32 bit tile into per-expert bitmaps with 32 ballots).  The CTA that finishes last (ticket
// counter) then scans: per expert the exclusive prefix over the blocks, and over the experts the
// exclusive prefix of the totals -> counts, offsets, n_sel.  Integer sums only: the result does
// not depend on which CTA is last.
__global__ void __launch_bounds__(TOKB)
bucket_count_scan_kernel(const uint32_t *__restrict__ mask, int T, int E, int W, int nblk,
                         int32_t *__restrict__ blockcounts, unsigned int *__restrict__ ticket,
                         int32_t *__restrict__ counts, int32_t *__restrict__ offsets, int32_t *__restrict__ n_sel,
                         int32_t *__restrict__ status, long long capacity)
{
    __shared__ int32_t cnt[TOKB / 32][33];
    __shared__ int warp_sums[8];
    __shared__ int chunk_total;
    __shared__ unsigned int my_ticket;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int t = blockIdx.x * TOKB + threadIdx.x;
    {
        const int w = blockIdx.y;                // one 32-expert mask word per CTA
        const uint32_t word = (t < T) ? __ldg(mask + (size_t)t * W + w) : 0u;
        cnt[warp][lane] = __popc(transpose_bits(word, lane));
        __syncthreads();
        if (warp == 0) {
            int total = 0;
#pragma unroll
            for (int i = 0; i < TOKB / 32; ++i) total += cnt[i][lane];
            const int e = w * 32 + lane;
            if (e < E) blockcounts[(size_t)blockIdx.x * E + e] = total;
        }
        __syncthreads();
    }
    __threadfence();
    if (threadIdx.x == 0) my_ticket = atomicAdd(ticket, 1u);
    __syncthreads();
    if (my_ticket != (unsigned int)(nblk * W - 1)) return;
    __threadfence();                         // every other CTA's block counts are visible now
    if (threadIdx.x == 0) *ticket = 0u;      // ready for the next call
    int carry = 0;
    for (int e0 = 0; e0 < E; e0 += TOKB) {
        const int e = e0 + threadIdx.x;
        int run = 0;
        if (e < E) {
            for (int b = 0; b < nblk; ++b) {
                const int c = __ldcg(blockcounts + (size_t)b * E + e);
                blockcounts[(size_t)b * E + e] = run;      // exclusive prefix over the token blocks
                run += c;
            }
            counts[e] = run;
        }
        const int ex = block_exscan_256(run, warp_sums, &chunk_total);
        if (e < E) offsets[e] = carry + ex;
        carry += chunk_total;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        offsets[E] = carry;
        *n_sel = carry;
        if ((long long)carry > capacity) atomicMax(status, (int32_t)D2D_ERR_CAPACITY);
    }
}

// Writes the per-expert token lists.  Position of token t in expert e's list = offsets[e]
// + tokens of earlier blocks + tokens of earlier warps of this block + tokens of lower lanes,
// so lists come out in ascending token order.  For each expert bit the lanes that hold it write
// consecutive entries (a coalesced store).
__global__ void __launch_bounds__(TOKB)
bucket_fill_kernel(const uint32_t *__restrict__ mask, int T, int E, int W,
                   const int32_t *__restrict__ blockbase, const int32_t *__restrict__ offsets,
                   int32_t *__restrict__ perm, long long capacity)
{
    __shared__ int32_t cnt[TOKB / 32][33];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int t = blockIdx.x * TOKB + threadIdx.x;
    const uint32_t lower = (1u << lane) - 1u;
    {
        const int w = blockIdx.y;                // one 32-expert mask word per CTA
        const int e = w * 32 + lane;
        // start of this CTA's run inside expert e's list (lane = expert); issued early to hide the latency
        const long long cta_base = e < E ? (long long)__ldg(offsets + e) + __ldg(blockbase + (size_t)blockIdx.x * E + e) : 0;
        const uint32_t word = (t < T) ? __ldg(mask + (size_t)t * W + w) : 0u;
        cnt[warp][lane] = __popc(transpose_bits(word, lane));
        __syncthreads();
        int before = 0;
        for (int i = 0; i < warp; ++i) before += cnt[i][lane];
        const long long base = cta_base + before;
#pragma unroll 4
        for (int j = 0; j < 32; ++j) {
            const uint32_t holders = __ballot_sync(FULL, (word >> j) & 1u);
            const long long bj = __shfl_sync(FULL, base, j);
            if ((word >> j) & 1u) {
                const long long idx = bj + __popc(holders & lower);
                if (idx < capacity) perm[idx] = t;
            }
        }
    }
}

// Exclusive scan of one int per thread over a 1024-thread CTA (used by the token-major dual).
__device__ __forceinline__ int block_exscan_1024(int v, int *warp_sums /*[32]*/, int *total_out)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int n = __shfl_up_sync(FULL, inc, o);
        if (lane >= o) inc += n;
    }
    if (lane == 31) warp_sums[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        const int ws = warp_sums[lane];
        int winc = ws;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int n = __shfl_up_sync(FULL, winc, o);
            if (lane >= o) winc += n;
        }
        warp_sums[lane] = winc - ws;
        if (lane == 31) *total_out = winc;
    }
    __syncthreads();
    const int res = warp_sums[warp] + inc - v;
    __syncthreads();
    return res;
}

// ---------------------------------------------------------------------------- token-major dual

__global__ void __launch_bounds__(1024)
tok_scan_kernel(const int32_t *__restrict__ k, int T, int32_t *__restrict__ tok_off)
{
    __shared__ int warp_sums[32];
    __shared__ int chunk_total;
    int carry = 0;
    for (int t0 = 0; t0 < T; t0 += 1024) {
        const int t = t0 + threadIdx.x;
        const int v = (t < T) ? k[t] : 0;
        const int ex = block_exscan_1024(v, warp_sums, &chunk_total);
        if (t < T) tok_off[t] = carry + ex;
        carry += chunk_total;
        __syncthreads();
    }
    if (threadIdx.x == 0) tok_off[T] = carry;
}

__global__ void __launch_bounds__(256)
tok_fill_kernel(const uint32_t *__restrict__ mask, int T, int W, const int32_t *__restrict__ tok_off,
                int32_t *__restrict__ tok_exp, long long capacity)
{
    const int lane = threadIdx.x & 31;
    const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (t >= T) return;
    long long base = tok_off[t];
    for (int w = 0; w < W; ++w) {
        const uint32_t word = __ldg(mask + (size_t)t * W + w);
        if ((word >> lane) & 1u) {
            const long long idx = base + __popc(word & ((1u << lane) - 1u));
            if (idx < capacity) tok_exp[idx] = w * 32 + lane;
        }
        base += __popc(word);
    }
}

}  // namespace

size_t d2d_select_ws_bytes(int T, int E)
{
    // [ticket counter, padded to 256 bytes | per-block, per-expert counters]
    const size_t nblk = (size_t)d2d_cdiv(T > 0 ? T : 1, TOKB);
    return 256 + d2d_align_up(nblk * (size_t)E * sizeof(int32_t), 256);
}

// Mask, k and status only (Eq. 4), T > 0; the sum of k is published through ksum (see the kernel).  The per-expert
// lists can be built afterwards, on any stream ordered behind this one, with d2d_launch_select(nullptr, ..., mask_ready = 1).
d2d_status d2d_launch_dynk_mask(const float *R, int T, int E, float tau, const d2d_routing *out, int32_t *ksum, cudaStream_t st)
{
    D2D_CUDA_TRY(cudaMemsetAsync(out->status, 0, sizeof(int32_t), st));
    dynk_mask_kernel<<<d2d_cdiv(T, 8), 256, 0, st>>>(R, T, E, (E + 31) / 32, tau, out->mask, out->k, out->status, ksum);
    D2D_LAUNCHED(1);
    return cudaGetLastError() == cudaSuccess ? D2D_OK : D2D_ERR_CUDA;
}

d2d_status d2d_launch_select(const float *R, int T, int E, float tau, int topk, const d2d_routing *out,
                             void *ws, cudaStream_t st, int mask_ready)
{
    const int W = (E + 31) / 32;
    if (!mask_ready) D2D_CUDA_TRY(cudaMemsetAsync(out->status, 0, sizeof(int32_t), st));
    if (T == 0) {
        D2D_CUDA_TRY(cudaMemsetAsync(out->counts, 0, sizeof(int32_t) * (size_t)E, st));
        D2D_CUDA_TRY(cudaMemsetAsync(out->offsets, 0, sizeof(int32_t) * (size_t)(E + 1), st));
        D2D_CUDA_TRY(cudaMemsetAsync(out->n_sel, 0, sizeof(int32_t), st));
        if (out->tok_off) D2D_CUDA_TRY(cudaMemsetAsync(out->tok_off, 0, sizeof(int32_t), st));
        return D2D_OK;
    }
    if (topk == 0 && d2d_small_select_supports(T, E)) return d2d_small_select(R, T, E, tau, out, st, mask_ready);
    const int warps_per_cta = 8;
    const int grid_tok = d2d_cdiv(T, warps_per_cta);
    if (R) {
        if (topk > 0)
            topk_mask_kernel<<<grid_tok, 256, 0, st>>>(R, T, E, W, topk, out->mask, out->k, out->status);
        else
            dynk_mask_kernel<<<grid_tok, 256, 0, st>>>(R, T, E, W, tau, out->mask, out->k, out->status, nullptr);
    } else if (!mask_ready) {
        k_from_mask_kernel<<<d2d_cdiv(T, 256), 256, 0, st>>>(out->mask, T, W, out->k);
    }
    const int nblk = d2d_cdiv(T, TOKB);
    unsigned int *ticket = (unsigned int *)ws;                    // must start at zero: cleared on every call
    int32_t *blockcounts = (int32_t *)((char *)ws + 256);
    D2D_CUDA_TRY(cudaMemsetAsync(ticket, 0, sizeof(unsigned int), st));
    bucket_count_scan_kernel<<<dim3(nblk, W), TOKB, 0, st>>>(out->mask, T, E, W, nblk, blockcounts, ticket, out->counts,
                                                    out->offsets, out->n_sel, out->status,
                                                    (long long)out->perm_capacity);
    bucket_fill_kernel<<<dim3(nblk, W), TOKB, 0, st>>>(out->mask, T, E, W, blockcounts, out->offsets, out->perm,
                                              (long long)out->perm_capacity);
    D2D_LAUNCHED(mask_ready ? 2 : 3);
    if (out->tok_off && out->tok_exp) {
        D2D_LAUNCHED(2);
        tok_scan_kernel<<<1, 1024, 0, st>>>(out->k, T, out->tok_off);
        tok_fill_kernel<<<grid_tok, 256, 0, st>>>(out->mask, T, W, out->tok_off, out->tok_exp,
                                                  (long long)out->perm_capacity);
    }
    return cudaGetLastError() == cudaSuccess ? D2D_OK : D2D_ERR_CUDA;
}

// ------------------------------------------------------------------------------------------
// d2d_select_dynk_static: the same selection + metadata, for callers that are not allowed to
// allocate device memory (and therefore cannot provide the workspace).  The per-block counter
// scratch lives in this file-scope device array instead.  Every GPU that loads the library
// holds these 512 KiB until the process exits.
//
// The name of a __device__ array is only a host-side stand-in in host code, not an address a
// kernel can use; the device address is fetched once per device with cudaGetSymbolAddress
// (with that device current) and cached.
// ------------------------------------------------------------------------------------------
#include <mutex>

#define D2D_STATIC_SCRATCH_INTS (128 * 1024)          /* 512 KiB: 64 + ceil(T/256) * E must not exceed this */
static __device__ __align__(256) int32_t d2d_select_static_scratch[D2D_STATIC_SCRATCH_INTS];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
int32_t *g_scratch_ptr[kMaxDevices] = {};
}

extern "C" D2D_API d2d_status d2d_select_dynk_static(const float *R, int32_t T, int32_t E, float tau,
                                                     d2d_routing *out, void *stream)
{
    if (T < 0 || E <= 0 || !out || !out->mask || !out->k || !out->counts || !out->offsets || !out->perm ||
        !out->n_sel || !out->status || out->perm_capacity < 0)
        return D2D_ERR_INVALID_ARG;
    if ((out->tok_off == nullptr) != (out->tok_exp == nullptr)) return D2D_ERR_INVALID_ARG;
    if (T > 0 && (!R || (reinterpret_cast<uintptr_t>(R) & 15u))) return D2D_ERR_INVALID_ARG;
    if (!(tau >= 0.0f && tau <= 1.0f)) return D2D_ERR_INVALID_ARG;
    // the scratch holds a ticket counter (64 ints reserved) and one counter per (block of 256 tokens, expert)
    const long long need = 64 + (long long)d2d_cdiv(T > 0 ? T : 1, TOKB) * (long long)E;
    if (need > (long long)D2D_STATIC_SCRATCH_INTS) return D2D_ERR_UNSUPPORTED;

    int dev = -1;
    D2D_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return D2D_ERR_UNSUPPORTED;
    int32_t *scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_scratch_mutex);
        if (!g_scratch_ptr[dev]) {
            // first call on this device: resolve the device address of the array (not capturable work)
            void *p = nullptr;
            if (cudaGetSymbolAddress(&p, d2d_select_static_scratch) != cudaSuccess || !p) return D2D_ERR_CUDA;
            g_scratch_ptr[dev] = static_cast<int32_t *>(p);
        }
        scratch = g_scratch_ptr[dev];
    }
    // the ticket counter at the front must start at zero and is cleared by the launch sequence on
    // every call; the block counters need no clearing (each is written before it is read)
    return d2d_launch_select(R, T, E, tau, 0, out, scratch, (cudaStream_t)stream);
}
