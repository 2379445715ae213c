// Selection for a small batch (T <= MAX_T; the stand-alone kernel takes up to 64 tokens) done by ONE CTA: row max, threshold, mask words, k, per-expert counts,
// offsets, token lists and the token-major dual.  Shared by the stand-alone selection kernel and by the
// small-batch router kernel, whose last CTA selects right after it has written the scores (one launch less
// on the decode path).  Dynamic-k rule: Sec. 3.4, Eq. 4 (keep expert i of token t when R[t,i] >= tau * max_j R[t,j]).
#pragma once

#include "d2d_common.cuh"

namespace d2d_small {

constexpr unsigned FULL = 0xffffffffu;
constexpr int MAX_T = 256;          // tokens select_cta can take (per-token k staged in shared memory)

__device__ __forceinline__ bool finite_f32(float v) { return (__float_as_uint(v) & 0x7f800000u) != 0x7f800000u; }

// Called by every thread of the CTA (blockDim.x a multiple of 32, at most 1024).  smask: shared memory, T * W words.
// R == nullptr: the mask words are an input (override protocol), otherwise they are computed.  R may have been
// written earlier by this very CTA (after a __syncthreads), hence the plain (coherent) loads.
__device__ __forceinline__ void select_cta(const float *R, int T, int E, int W, float tau, uint32_t *mask, int32_t *k,
                                           int32_t *counts, int32_t *offsets, int32_t *perm, int32_t *tok_off,
                                           int32_t *tok_exp, int32_t *n_sel, int32_t *status, long long capacity,
                                           int keep_status, uint32_t *smask)
{
    __shared__ int warp_sums[32];
    __shared__ int chunk_total;
    __shared__ int sk[MAX_T];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int nthreads = blockDim.x, nwarps = nthreads >> 5;
    if (threadIdx.x == 0 && !keep_status) *status = 0;
    __syncthreads();

    for (int t = warp; t < T; t += nwarps) {
        int kt = 0;
        if (R) {
            const float *row = R + (size_t)t * E;
            float m = -INFINITY;
            bool bad = false;
            for (int i = lane; i < E; i += 32) {
                const float v = row[i];
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
                const bool keep = (i < E) && (bad || row[i] >= thr);
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

    // per-expert counts, the exclusive scan over experts and the token lists
    int carry = 0;
    if (E * 4 <= nthreads) {
        // few experts: a warp per expert with its lanes over the tokens (ballots keep the lists in ascending order)
        __shared__ int scnt[256], soff[256];
        const uint32_t lower = (1u << lane) - 1u;
        for (int e = warp; e < E; e += nwarps) {
            int c = 0;
            for (int t0 = 0; t0 < T; t0 += 32) {
                const int t = t0 + lane;
                const bool bit = t < T && ((smask[t * W + (e >> 5)] >> (e & 31)) & 1u);
                c += __popc(__ballot_sync(FULL, bit));
            }
            if (lane == 0) scnt[e] = c;
        }
        __syncthreads();
        if (warp == 0) {
            int run = 0;
            for (int e0 = 0; e0 < E; e0 += 32) {
                const int e = e0 + lane;
                const int c = e < E ? scnt[e] : 0;
                int inc = c;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int n = __shfl_up_sync(FULL, inc, o);
                    if (lane >= o) inc += n;
                }
                if (e < E) {
                    soff[e] = run + inc - c;
                    counts[e] = c;
                    offsets[e] = run + inc - c;
                }
                run += __shfl_sync(FULL, inc, 31);
            }
            if (lane == 0) chunk_total = run;
        }
        __syncthreads();
        carry = chunk_total;
        for (int e = warp; e < E; e += nwarps) {
            long long idx = soff[e];
            for (int t0 = 0; t0 < T; t0 += 32) {
                const int t = t0 + lane;
                const bool bit = t < T && ((smask[t * W + (e >> 5)] >> (e & 31)) & 1u);
                const uint32_t b = __ballot_sync(FULL, bit);
                const long long at = idx + __popc(b & lower);
                if (bit && at < capacity) perm[at] = t;
                idx += __popc(b);
            }
        }
    } else {
    for (int e0 = 0; e0 < E; e0 += nthreads) {
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
            const int ws = lane < nwarps ? warp_sums[lane] : 0;
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
    }
    if (threadIdx.x == 0) {
        offsets[E] = carry;
        *n_sel = carry;
        if ((long long)carry > capacity) atomicMax(status, (int32_t)D2D_ERR_CAPACITY);
    }
    // token-major dual: exclusive scan of k by warp 0, then one thread per token
    if (tok_off && tok_exp) {
        __shared__ int stok[MAX_T];
        __syncthreads();
        if (warp == 0) {
            int run = 0;
            for (int t0 = 0; t0 < T; t0 += 32) {
                const int t = t0 + lane;
                const int c = t < T ? sk[t] : 0;
                int inc = c;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int n = __shfl_up_sync(FULL, inc, o);
                    if (lane >= o) inc += n;
                }
                if (t < T) stok[t] = run + inc - c;
                run += __shfl_sync(FULL, inc, 31);
            }
        }
        __syncthreads();
        for (int t = threadIdx.x; t < T; t += nthreads) {
            long long base = stok[t];
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
}

}  // namespace d2d_small
