// Small-batch (decode) path: T <= 64 tokens.  Here the layer is bound by HBM traffic and by launch
// latency, not by arithmetic: every selected expert's weight slice is read exactly once, with
// 16-byte loads, by a CTA of its own, and the number of launches is kept to a minimum.
//
//   small_select_kernel   one CTA does the whole selection: row max, threshold, mask words, k,
//                         per-expert counts, offsets, token lists (and the token-major dual)
// The router and expert kernels of this path are in small_batch_ffn.cu.
#include "d2d_common.cuh"

namespace {

constexpr unsigned FULL = 0xffffffffu;

__device__ __forceinline__ bool finite_f32(float v) { return (__float_as_uint(v) & 0x7f800000u) != 0x7f800000u; }

// ------------------------------------------------------------------------------------ selection

// R == nullptr: the mask words are an input (override protocol), otherwise they are computed.
__global__ void __launch_bounds__(1024)
small_select_kernel(const float *__restrict__ R, int T, int E, int W, float tau,
                    uint32_t *__restrict__ mask, int32_t *__restrict__ k, int32_t *__restrict__ counts,
                    int32_t *__restrict__ offsets, int32_t *__restrict__ perm, int32_t *__restrict__ tok_off,
                    int32_t *__restrict__ tok_exp, int32_t *__restrict__ n_sel, int32_t *__restrict__ status,
                    long long capacity, int keep_status)
{
    extern __shared__ uint32_t smask[];          // [T][W]
    __shared__ int warp_sums[32];
    __shared__ int chunk_total;
    __shared__ int sk[64];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0 && !keep_status) *status = 0;
    __syncthreads();

    for (int t = warp; t < T; t += 32) {
        int kt = 0;
        if (R) {
            const float *row = R + (size_t)t * E;
            float m = -INFINITY;
            bool bad = false;
            for (int i = lane; i < E; i += 32) {
                const float v = __ldg(row + i);
                bad |= !finite_f32(v);
                m = v > m ? v : m;
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float other = __shfl_xor_sync(FULL, m, o);
                m = other > m ? other : m;
            }
            bad = __any_sync(FULL, bad);
            const float thr = __fmul_rn(tau, m);
            for (int w = 0; w < W; ++w) {
                const int i = w * 32 + lane;
                const bool keep = (i < E) && (bad || __ldg(row + i) >= thr);
                const uint32_t word = __ballot_sync(FULL, keep);
                if (lane == 0) { mask[(size_t)t * W + w] = word; smask[t * W + w] = word; }
                kt += __popc(word);
            }
            if (lane == 0 && bad) atomicMax(status, (int32_t)D2D_ERR_NONFINITE);
        } else {
            for (int w = lane; w < W; w += 32) {
                const uint32_t word = mask[(size_t)t * W + w];
                smask[t * W + w] = word;
                kt += __popc(word);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) kt += __shfl_xor_sync(FULL, kt, o);
        }
        if (lane == 0) { k[t] = kt; sk[t] = kt; }
    }
    __syncthreads();

    // per-expert counts and the exclusive scan over experts (chunks of 1024 experts)
    int carry = 0;
    for (int e0 = 0; e0 < E; e0 += 1024) {
        const int e = e0 + threadIdx.x;
        int c = 0;
        if (e < E)
            for (int t = 0; t < T; ++t) c += (smask[t * W + (e >> 5)] >> (e & 31)) & 1u;
        // block-wide exclusive scan of c
        int inc = c;
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
            if (lane == 31) chunk_total = winc;
        }
        __syncthreads();
        const int off = carry + warp_sums[warp] + inc - c;
        if (e < E) {
            counts[e] = c;
            offsets[e] = off;
            long long idx = off;
            for (int t = 0; t < T; ++t)
                if ((smask[t * W + (e >> 5)] >> (e & 31)) & 1u) {
                    if (idx < capacity) perm[idx] = t;
                    ++idx;
                }
        }
        carry += chunk_total;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        offsets[E] = carry;
        *n_sel = carry;
        if ((long long)carry > capacity) atomicMax(status, (int32_t)D2D_ERR_CAPACITY);
    }
    // token-major dual: T <= 64, one thread per token
    if (tok_off && tok_exp && threadIdx.x < T) {
        const int t = threadIdx.x;
        long long base = 0;
        for (int u = 0; u < t; ++u) base += sk[u];
        tok_off[t] = (int32_t)base;
        if (t == T - 1) tok_off[T] = (int32_t)(base + sk[t]);
        for (int w = 0; w < W; ++w) {
            uint32_t word = smask[t * W + w];
            while (word) {
                const int b = __ffs(word) - 1;
                word &= word - 1;
                if (base < capacity) tok_exp[base] = w * 32 + b;
                ++base;
            }
        }
    }
}

}  // namespace

bool d2d_small_select_supports(int T, int E) { return T >= 1 && T <= 64 && (size_t)T * ((E + 31) / 32) * 4 <= 96 * 1024; }

d2d_status d2d_small_select(const float *R, int T, int E, float tau, const d2d_routing *out, cudaStream_t st,
                            int mask_ready)
{
    const int W = (E + 31) / 32;
    const size_t smem = (size_t)T * W * sizeof(uint32_t);
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(small_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024) != cudaSuccess)
            return D2D_ERR_CUDA;
        attr_set = true;
    }
    small_select_kernel<<<1, 1024, smem, st>>>(R, T, E, W, tau, out->mask, out->k, out->counts, out->offsets, out->perm,
                                               out->tok_off, out->tok_exp, out->n_sel, out->status,
                                               (long long)out->perm_capacity, mask_ready);
    D2D_LAUNCHED(1);
    return cudaGetLastError() == cudaSuccess ? D2D_OK : D2D_ERR_CUDA;
}

