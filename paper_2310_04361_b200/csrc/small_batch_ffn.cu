// Small-batch (decode) router and expert kernels: T <= 64 tokens, bound by HBM traffic and latency.
//
// Both kernels bring every weight byte they need into shared memory with 16-byte cp.async copies
// that are all issued before the first use (maximum memory-level parallelism: the copies of a CTA
// are in flight together instead of one cache line at a time), then compute from shared memory.
//
//   small_router_kernel   CTA b owns 8 hidden units: its 8 rows of W_r1 and all token rows go to
//                         shared memory, one warp per unit forms u[t, j]; every CTA also prefetches
//                         W_r2, and the CTA that finishes last (ticket) computes layer 2 from it and,
//                         when asked to, the dynamic-k selection and its metadata as well (no second launch)
//   small_ffn_kernel      one CTA per expert (several for experts too large for one pass): the W1 / W_gate / W2 slices are read from HBM exactly
//                         once (only experts some token kept do any work), the expert's tokens are
//                         handled 8 at a time, partial output rows go to a float32 accumulator with
//                         16-byte vector reductions; the last CTA adds b2 and writes y
#include <cuda_fp8.h>
#include <type_traits>

#include "d2d_common.cuh"
#include "small_select.cuh"

namespace {

constexpr int MAX_TBLK = 8;        // at most this many tokens are processed together (template parameter TBLK)
constexpr int NT = 256;

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(void *dst_smem, const void *src_gmem)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_addr(dst_smem)), "l"(src_gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Copies `bytes` (multiple of 16, both sides 16-byte aligned) with every thread of the CTA.
__device__ __forceinline__ void cta_copy_async(void *dst_smem, const void *src_gmem, size_t bytes)
{
    for (size_t off = (size_t)threadIdx.x * 16; off < bytes; off += (size_t)NT * 16)
        cp_async16((char *)dst_smem + off, (const char *)src_gmem + off);
}

// 8 consecutive elements from shared memory as floats
__device__ __forceinline__ void lds8(const float *p, float (&o)[8])
{
    const float4 a = *reinterpret_cast<const float4 *>(p), b = *(reinterpret_cast<const float4 *>(p) + 1);
    o[0] = a.x; o[1] = a.y; o[2] = a.z; o[3] = a.w; o[4] = b.x; o[5] = b.y; o[6] = b.z; o[7] = b.w;
}
__device__ __forceinline__ void lds8(const __nv_bfloat16 *p, float (&o)[8])
{
    const uint4 raw = *reinterpret_cast<const uint4 *>(p);
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        o[2 * i] = __uint_as_float(w[i] << 16);
        o[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}

// 8 consecutive 8-bit floating point codes (e4m3) as floats; the expert's power-of-two scale is applied by the caller
__device__ __forceinline__ void lds8(const uint8_t *p, float (&o)[8])
{
    const uint2 raw = *reinterpret_cast<const uint2 *>(p);
    const uint32_t w[2] = {raw.x, raw.y};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const __half2_raw h = __nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)((w[i >> 1] >> ((i & 1) * 16)) & 0xffffu), __NV_E4M3);
        const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&h));
        o[2 * i] = f.x;
        o[2 * i + 1] = f.y;
    }
}

// One warp: dot products of a weight row with up to TBLK token rows, all operands in shared memory.
template <typename WT, typename TT, int TBLK>
__device__ __forceinline__ void warp_row_dots(const WT *wrow, const TT *xs, int d, int lane, float (&acc)[TBLK])
{
#pragma unroll
    for (int i = 0; i < TBLK; ++i) acc[i] = 0.0f;
    for (int c = lane * 8; c < d; c += 256) {
        float wv[8];
        lds8(wrow + c, wv);
#pragma unroll
        for (int i = 0; i < TBLK; ++i) {
            float xv[8];
            lds8(xs + (size_t)i * d + c, xv);
#pragma unroll
            for (int q = 0; q < 8; ++q) acc[i] = fmaf(wv[q], xv[q], acc[i]);
        }
    }
#pragma unroll
    for (int i = 0; i < TBLK; ++i) acc[i] = d2d_warp_sum(acc[i]);
}

// ------------------------------------------------------------------------------------ router

// Outputs of the selection the router's last CTA may perform (enabled == 0: scores only).
struct SmallSel {
    int enabled;
    float tau;
    uint32_t *mask;
    int32_t *k, *counts, *offsets, *perm, *tok_off, *tok_exp, *n_sel, *status;
    long long capacity;
};

// Per-layer arguments; blockIdx.y picks the layer, so that several layers of one shape that read the same tokens
// (the Q, K and V projections of an attention layer) run as one grid.
struct SmallRouterLayer {
    const void *w_r1, *b_r1, *w_r2, *b_r2;
    float *u, *R;
    unsigned int *ticket;
    float *zero;
    SmallSel sel;
};
struct SmallRouterArgs {
    SmallRouterLayer l[D2D_MAX_GROUP];
};

// dynamic shared memory: [ W_r1 rows of this CTA: 8*d | token block: TBLK*d | W_r2: E*d_h (if staged) | u: T*d_h floats |
//                          selection words: T*ceil(E/32) ]
template <typename TT, int TBLK>
__global__ void __launch_bounds__(NT)
small_router_kernel(const TT *__restrict__ x, int T, int d, int d_h, int E, int stage_w2, int zero_words,
                    const __grid_constant__ SmallRouterArgs args)
{
    const SmallRouterLayer &P = args.l[blockIdx.y];
    const TT *__restrict__ w_r1 = static_cast<const TT *>(P.w_r1);
    const TT *__restrict__ b_r1 = static_cast<const TT *>(P.b_r1);
    const TT *__restrict__ w_r2 = static_cast<const TT *>(P.w_r2);
    const TT *__restrict__ b_r2 = static_cast<const TT *>(P.b_r2);
    float *__restrict__ u = P.u;
    float *R = P.R;
    unsigned int *__restrict__ ticket = P.ticket;
    float *__restrict__ zero = P.zero;
    const SmallSel &sel = P.sel;
    // clear the float32 accumulator of the expert kernel that follows on the stream (saves a memset node)
    for (int i = blockIdx.x * NT + threadIdx.x; i < zero_words; i += gridDim.x * NT) zero[i] = 0.0f;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    TT *w1s = reinterpret_cast<TT *>(smem_raw);
    TT *xs = w1s + (size_t)8 * d;
    TT *w2s = xs + (size_t)TBLK * d;
    // W_r2 rows are staged with a pitch of d_h + 16 bytes: in layer 2 each thread walks its own row, and with the
    // natural pitch (a multiple of 128 bytes) all lanes of a warp would hit the same shared-memory banks
    const int w2_pitch = d_h + (int)(16 / sizeof(TT));
    float *us = reinterpret_cast<float *>(w2s + (stage_w2 ? (size_t)E * w2_pitch : 0));
    __shared__ unsigned int my_ticket;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int j0 = blockIdx.x * 8;
    const int rows = d_h - j0 < 8 ? d_h - j0 : 8;

    // copy groups: [W_r1 rows + first token block] first, W_r2 (needed only by the last CTA, prefetched by all) second,
    // so that layer 1 starts as soon as its own operands have landed and does not wait for the 2*E*d_h bytes of W_r2
    cta_copy_async(w1s, w_r1 + (size_t)j0 * d, (size_t)rows * d * sizeof(TT));
    {
        const int ntok0 = T < TBLK ? T : TBLK;
        cta_copy_async(xs, x, (size_t)ntok0 * d * sizeof(TT));
    }
    cp_async_commit();
    if (stage_w2) {
        const int cpr = d_h * (int)sizeof(TT) / 16;               // 16-byte chunks per row
        for (int c = threadIdx.x; c < E * cpr; c += NT) {
            const int row = c / cpr, w = c - row * cpr;
            cp_async16(reinterpret_cast<char *>(w2s + (size_t)row * w2_pitch) + w * 16,
                       reinterpret_cast<const char *>(w_r2 + (size_t)row * d_h) + w * 16);
        }
    }
    cp_async_commit();

    for (int t0 = 0; t0 < T; t0 += TBLK) {
        const int ntok = T - t0 < TBLK ? T - t0 : TBLK;
        if (t0 > 0) {
            __syncthreads();                                      // previous block's readers of xs are done
            cta_copy_async(xs, x + (size_t)t0 * d, (size_t)ntok * d * sizeof(TT));
            cp_async_commit();
        }
        if (ntok < TBLK)                                          // unused token slots read zeros
            for (int i = threadIdx.x; i < (TBLK - ntok) * d; i += NT) xs[(size_t)ntok * d + i] = d2d_from_float<TT>(0.0f);
        if (t0 == 0) cp_async_wait<1>();                          // the first group: W_r1 rows and the first token block
        else cp_async_wait<0>();
        __syncthreads();
        if (warp < rows) {
            float acc[TBLK];
            warp_row_dots<TT, TT, TBLK>(w1s + (size_t)warp * d, xs, d, lane, acc);
            if (lane == 0) {
                const float bj = b_r1 ? d2d_to_float<TT>(b_r1[j0 + warp]) : 0.0f;
#pragma unroll
                for (int i = 0; i < TBLK; ++i)
                    if (i < ntok) u[(size_t)(t0 + i) * d_h + j0 + warp] = fmaxf(acc[i] + bj, 0.0f);
            }
        }
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) my_ticket = atomicAdd(ticket, 1u);
    __syncthreads();
    if (my_ticket != gridDim.x - 1) {
        cp_async_wait<0>();                                       // no copy may be in flight when the CTA exits
        return;
    }
    __threadfence();
    if (threadIdx.x == 0) *ticket = 0u;
    // ---- layer 2 by the last CTA: a thread owns an expert, keeps TBLK accumulators, walks its W_r2 row
    for (int i = threadIdx.x; i < T * d_h; i += NT) us[i] = __ldcg(u + i);
    cp_async_wait<0>();
    __syncthreads();
    for (int i = threadIdx.x; i < E; i += NT) {
        const float bi = b_r2 ? d2d_to_float<TT>(b_r2[i]) : 0.0f;
        for (int t0 = 0; t0 < T; t0 += TBLK) {
            float acc[TBLK];
#pragma unroll
            for (int q = 0; q < TBLK; ++q) acc[q] = 0.0f;
            for (int c = 0; c < d_h; c += 8) {
                float wv[8];
                if (stage_w2) lds8(w2s + (size_t)i * w2_pitch + c, wv);
                else d2d_load8(w_r2 + (size_t)i * d_h + c, wv);
#pragma unroll
                for (int q = 0; q < TBLK; ++q) {
                    const float *ur = us + (size_t)(t0 + q < T ? t0 + q : t0) * d_h + c;
#pragma unroll
                    for (int z = 0; z < 8; ++z) acc[q] = fmaf(wv[z], ur[z], acc[q]);
                }
            }
#pragma unroll
            for (int q = 0; q < TBLK; ++q)
                if (t0 + q < T) R[(size_t)(t0 + q) * E + i] = fabsf(acc[q] + bi);
        }
    }
    if (sel.enabled) {
        // the scores of all (at most 8) tokens were written by this CTA: select from them right here
        __syncthreads();
        uint32_t *smask = reinterpret_cast<uint32_t *>(us + (size_t)T * d_h);
        d2d_small::select_cta(R, T, E, (E + 31) / 32, sel.tau, sel.mask, sel.k, sel.counts, sel.offsets, sel.perm, sel.tok_off,
                              sel.tok_exp, sel.n_sel, sel.status, sel.capacity, 0, smask);
    }
}

// ------------------------------------------------------------------------------------ expert FFN

__device__ __forceinline__ void red_add_v4(float *addr, float a, float b, float c, float d)
{
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}

// dynamic shared memory: [ W1 rows: rc*d | W_gate rows: rc*d (gated) | W2T rows: rc*d | token block: TBLK*d | h: TBLK*rc floats ]
// rc = neurons handled per pass (the whole expert when its slices fit).
struct SmallFfnLayer {
    const void *w1, *b1, *w_gate, *w2t, *b2;   // Q8 kernels: w1, w_gate, w2t are e4m3 codes [d_ff, d]
    const int32_t *offsets, *perm;
    float *y32;
    unsigned int *ticket;
    void *y;
    long long capacity;      // entries the caller's perm buffer holds: a list truncated by D2D_ERR_CAPACITY is never read past it
    const int32_t *k1, *kg, *k2;      // Q8 kernels: per-expert exponents of the scales 2^k of W1, W_gate, W2
};
struct SmallFfnArgs {
    SmallFfnLayer l[D2D_MAX_GROUP];
};

// Q8: the expert weights are 8-bit floating point codes (e4m3) with one power-of-two scale per expert and matrix
// (App. C runs the expert kernels on narrower formats): half the bytes per kept expert; the codes are widened when they
// are used and the scale, a power of two, is applied to the finished sums (exactly what scaling every weight would give).
template <typename TT, int ACT, bool GATED, int TBLK, bool Q8>
__global__ void __launch_bounds__(NT)
small_ffn_kernel(const TT *__restrict__ x, int T, int d, int s, int rc, int splits, const __grid_constant__ SmallFfnArgs args)
{
    using WT = typename std::conditional<Q8, uint8_t, TT>::type;
    const SmallFfnLayer &P = args.l[blockIdx.y];
    const WT *__restrict__ w1 = static_cast<const WT *>(P.w1);
    const TT *__restrict__ b1 = static_cast<const TT *>(P.b1);
    const WT *__restrict__ w_gate = static_cast<const WT *>(P.w_gate);
    const WT *__restrict__ w2t = static_cast<const WT *>(P.w2t);
    const TT *__restrict__ b2 = static_cast<const TT *>(P.b2);
    const int32_t *__restrict__ offsets = P.offsets;
    const int32_t *__restrict__ perm = P.perm;
    float *__restrict__ y32 = P.y32;
    unsigned int *__restrict__ ticket = P.ticket;
    TT *__restrict__ y = static_cast<TT *>(P.y);
    extern __shared__ __align__(16) unsigned char smem_raw[];
    WT *w1s = reinterpret_cast<WT *>(smem_raw);
    WT *wgs = w1s + (size_t)rc * d;
    WT *w2s = wgs + (GATED ? (size_t)rc * d : 0);
    TT *xs = reinterpret_cast<TT *>(w2s + (size_t)rc * d);
    float *hs = reinterpret_cast<float *>(xs + (size_t)TBLK * d);
    __shared__ unsigned int my_ticket;
    __shared__ int stok[TBLK];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // an expert too large for one pass is shared by `splits` CTAs, each with its own range of neurons (one pass of rc
    // neurons when splits = ceil(s / rc)): the kept experts then fill the machine instead of a fraction of its SMs
    const int e = blockIdx.x / splits, part = blockIdx.x - e * splits;
    const int span = ((s + splits - 1) / splits + rc - 1) / rc * rc, r_begin = part * span, r_end = r_begin + span < s ? r_begin + span : s;
    const float sc1 = Q8 ? ldexpf(1.0f, P.k1[e]) : 1.0f, scg = Q8 && GATED ? ldexpf(1.0f, P.kg[e]) : 1.0f, sc2 = Q8 ? ldexpf(1.0f, P.k2[e]) : 1.0f;
    // perm may have been truncated at `capacity` entries (the selection then reported D2D_ERR_CAPACITY): stay inside it
    const long long cap = P.capacity;
    const int end = (long long)offsets[e + 1] < cap ? offsets[e + 1] : (int)cap;
    const int beg = offsets[e] < end ? offsets[e] : end;

    if (beg < end) {
        for (int r0 = r_begin; r0 < r_end; r0 += rc) {
            const int rows = r_end - r0 < rc ? r_end - r0 : rc;
            const size_t n0 = (size_t)e * s + r0;
            __syncthreads();                                      // readers of the previous pass are done
            cta_copy_async(w1s, w1 + n0 * d, (size_t)rows * d * sizeof(WT));
            if (GATED) cta_copy_async(wgs, w_gate + n0 * d, (size_t)rows * d * sizeof(WT));
            cta_copy_async(w2s, w2t + n0 * d, (size_t)rows * d * sizeof(WT));
            cp_async_commit();
            for (int p0 = beg; p0 < end; p0 += TBLK) {
                const int ntok = end - p0 < TBLK ? end - p0 : TBLK;
                __syncthreads();                                  // previous token block fully consumed
                if (threadIdx.x < TBLK) {
                    const int tok = perm[p0 + (threadIdx.x < ntok ? threadIdx.x : 0)];
                    stok[threadIdx.x] = tok < 0 ? 0 : tok >= T ? T - 1 : tok;      // a corrupt list cannot address outside x and y
                }
                __syncthreads();
                for (int i = 0; i < ntok; ++i) cta_copy_async(xs + (size_t)i * d, x + (size_t)stok[i] * d, (size_t)d * sizeof(TT));
                if (ntok < TBLK)
                    for (int i = threadIdx.x; i < (TBLK - ntok) * d; i += NT) xs[(size_t)ntok * d + i] = d2d_from_float<TT>(0.0f);
                cp_async_commit();
                cp_async_wait<0>();
                __syncthreads();
                // ---- up projection + activation: one warp per neuron
                for (int nl = warp; nl < rows; nl += NT / 32) {
                    float up[TBLK], gate[TBLK];
                    warp_row_dots<WT, TT, TBLK>(w1s + (size_t)nl * d, xs, d, lane, up);
                    if (GATED) warp_row_dots<WT, TT, TBLK>(wgs + (size_t)nl * d, xs, d, lane, gate);
                    if (lane == 0) {
                        const float bn = b1 ? d2d_to_float<TT>(b1[n0 + nl]) : 0.0f;
#pragma unroll
                        for (int i = 0; i < TBLK; ++i) {
                            const float z = up[i] * sc1 + bn;
                            hs[i * rc + nl] = GATED ? d2d_activate<ACT>(gate[i] * scg) * z : d2d_activate<ACT>(z);
                        }
                    }
                }
                __syncthreads();
                // ---- down projection: a thread owns 4 adjacent output columns
                for (int c = threadIdx.x * 4; c < d; c += NT * 4) {
                    float acc[TBLK][4];
#pragma unroll
                    for (int i = 0; i < TBLK; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.0f;
                    for (int nl = 0; nl < rows; ++nl) {
                        const WT *wp = w2s + (size_t)nl * d + c;
                        float w0, w1v, w2v, w3;
                        if (Q8) {
                            const uint32_t raw = *reinterpret_cast<const uint32_t *>(wp);
                            const __half2_raw lo = __nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)(raw & 0xffffu), __NV_E4M3);
                            const __half2_raw hi = __nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)(raw >> 16), __NV_E4M3);
                            const float2 a = __half22float2(*reinterpret_cast<const __half2 *>(&lo));
                            const float2 b = __half22float2(*reinterpret_cast<const __half2 *>(&hi));
                            w0 = a.x; w1v = a.y; w2v = b.x; w3 = b.y;
                        } else if (sizeof(TT) == 2) {
                            const uint2 raw = *reinterpret_cast<const uint2 *>(wp);
                            w0 = __uint_as_float(raw.x << 16); w1v = __uint_as_float(raw.x & 0xffff0000u);
                            w2v = __uint_as_float(raw.y << 16); w3 = __uint_as_float(raw.y & 0xffff0000u);
                        } else {
                            const float4 raw = *reinterpret_cast<const float4 *>(wp);
                            w0 = raw.x; w1v = raw.y; w2v = raw.z; w3 = raw.w;
                        }
#pragma unroll
                        for (int i = 0; i < TBLK; ++i) {
                            const float h = hs[i * rc + nl];
                            acc[i][0] = fmaf(h, w0, acc[i][0]);
                            acc[i][1] = fmaf(h, w1v, acc[i][1]);
                            acc[i][2] = fmaf(h, w2v, acc[i][2]);
                            acc[i][3] = fmaf(h, w3, acc[i][3]);
                        }
                    }
#pragma unroll
                    for (int i = 0; i < TBLK; ++i)
                        if (i < ntok)
                            red_add_v4(y32 + (size_t)stok[i] * d + c, acc[i][0] * sc2, acc[i][1] * sc2, acc[i][2] * sc2, acc[i][3] * sc2);
                }
            }
        }
    }
    // ---- the CTA that finishes last converts the float32 accumulator (+ b2) to the output dtype
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) my_ticket = atomicAdd(ticket, 1u);
    __syncthreads();
    if (my_ticket != gridDim.x - 1) return;
    __threadfence();
    if (threadIdx.x == 0) *ticket = 0u;
    const size_t total = (size_t)T * d;
    for (size_t i = (size_t)threadIdx.x * 4; i < total; i += (size_t)NT * 4) {
        const float4 v = __ldcg(reinterpret_cast<const float4 *>(y32 + i));
        const int c = (int)(i % d);
        float o[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int q = 0; q < 4; ++q) y[i + q] = d2d_from_float<TT>(o[q] + (b2 ? d2d_to_float<TT>(b2[c + q]) : 0.0f));
    }
}

constexpr size_t kSmemLimit = 200 * 1024;

// neurons per pass so that the slices, one token block and the hidden values fit in shared memory
int rows_per_pass(const d2d_layer_desc &D, size_t elem, int tb = MAX_TBLK, size_t welem = 0)
{
    if (welem == 0) welem = elem;                              // weights stored like the activations unless stated
    const size_t n_mat = D.gated ? 3 : 2;
    const size_t fixed = (size_t)tb * D.d * elem;
    for (int rc = D.expert_size; rc >= 1; rc = (rc + 1) / 2) {
        const size_t need = n_mat * rc * D.d * welem + fixed + (size_t)tb * rc * 4;
        if (need <= kSmemLimit) return rc;
        if (rc == 1) break;
    }
    return 0;
}

// tokens handled together: the smallest of 1, 2, 4, 8 that covers the batch (a token slot that stays empty
// still costs its share of the dot products)
int token_block(int T) { return T <= 1 ? 1 : T <= 2 ? 2 : T <= 4 ? 4 : 8; }

template <typename TT, int ACT, bool GATED, int TBLK, bool Q8>
d2d_status launch_ffn_q(const d2d_layer_desc &D, int n_layers, const SmallFfnArgs &args, const void *x, int T, cudaStream_t st)
{
    const size_t welem = Q8 ? 1 : sizeof(TT);
    const int rc = rows_per_pass(D, sizeof(TT), TBLK, welem);
    if (rc <= 0) return D2D_ERR_UNSUPPORTED;
    const size_t smem = (size_t)(GATED ? 3 : 2) * rc * D.d * welem + (size_t)TBLK * D.d * sizeof(TT) + (size_t)TBLK * rc * 4;
    auto kern = small_ffn_kernel<TT, ACT, GATED, TBLK, Q8>;
    static size_t attr_smem = 0;
    if (smem > attr_smem) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemLimit) != cudaSuccess) return D2D_ERR_CUDA;
        attr_smem = kSmemLimit;
    }
    // a single token: one pass per CTA for experts that need several (measured on the Llama-shaped layer: 86 -> 82 us at
    // one token, but 108 -> 117 us at two, where every extra CTA stages the token rows and merges its partial sums again)
    const int splits = T == 1 ? d2d_cdiv(D.expert_size, rc) : 1;
    kern<<<dim3(D.n_experts * splits, n_layers), NT, smem, st>>>((const TT *)x, T, D.d, D.expert_size, rc, splits, args);
    D2D_LAUNCHED(1);
    return cudaGetLastError() == cudaSuccess ? D2D_OK : D2D_ERR_CUDA;
}

template <typename TT, int ACT, bool GATED, int TBLK>
d2d_status launch_ffn_tb(const d2d_layer_desc &D, int n_layers, const SmallFfnArgs &args, const void *x, int T, cudaStream_t st)
{
    // 8-bit weights: bf16 layers only (one layer per launch: every layer of the launch must hold codes)
    if (std::is_same<TT, __nv_bfloat16>::value && n_layers == 1 && args.l[0].k1 != nullptr)
        return launch_ffn_q<TT, ACT, GATED, TBLK, std::is_same<TT, __nv_bfloat16>::value>(D, n_layers, args, x, T, st);
    return launch_ffn_q<TT, ACT, GATED, TBLK, false>(D, n_layers, args, x, T, st);
}

template <typename TT, int ACT, bool GATED>
d2d_status launch_ffn(const d2d_layer_desc &D, int n, const SmallFfnArgs &a, const void *x, int T, cudaStream_t st)
{
    switch (token_block(T)) {
    case 1: return launch_ffn_tb<TT, ACT, GATED, 1>(D, n, a, x, T, st);
    case 2: return launch_ffn_tb<TT, ACT, GATED, 2>(D, n, a, x, T, st);
    case 4: return launch_ffn_tb<TT, ACT, GATED, 4>(D, n, a, x, T, st);
    default: return launch_ffn_tb<TT, ACT, GATED, 8>(D, n, a, x, T, st);
    }
}

template <typename TT, int ACT>
d2d_status launch_ffn_gated(const d2d_layer_desc &D, int n, const SmallFfnArgs &a, const void *x, int T, cudaStream_t st)
{
    if (D.gated) return launch_ffn<TT, ACT, true>(D, n, a, x, T, st);
    return launch_ffn<TT, ACT, false>(D, n, a, x, T, st);
}

template <typename TT>
d2d_status launch_ffn_dtype(const d2d_layer_desc &D, int n, const SmallFfnArgs &a, const void *x, int T, cudaStream_t st)
{
    switch (D.act) {
    case D2D_ACT_RELU: return launch_ffn_gated<TT, D2D_ACT_RELU>(D, n, a, x, T, st);
    case D2D_ACT_GELU_ERF: return launch_ffn_gated<TT, D2D_ACT_GELU_ERF>(D, n, a, x, T, st);
    case D2D_ACT_GELU_TANH: return launch_ffn_gated<TT, D2D_ACT_GELU_TANH>(D, n, a, x, T, st);
    default: return launch_ffn_gated<TT, D2D_ACT_SILU>(D, n, a, x, T, st);
    }
}

template <typename TT, int TBLK>
d2d_status launch_router_tb(const d2d_layer_desc &D, int n_layers, const SmallRouterArgs &args, const void *x, int T,
                            int zero_words, cudaStream_t st)
{
    const size_t base = (size_t)(8 + TBLK) * D.d * sizeof(TT) + (size_t)T * D.d_h * 4 + (size_t)T * ((D.n_experts + 31) / 32) * 4;
    const size_t w2_bytes = (size_t)D.n_experts * (D.d_h * sizeof(TT) + 16);      // padded pitch, see the kernel
    const int stage_w2 = base + w2_bytes <= kSmemLimit ? 1 : 0;
    const size_t smem = base + (stage_w2 ? w2_bytes : 0);
    auto kern = small_router_kernel<TT, TBLK>;
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemLimit) != cudaSuccess) return D2D_ERR_CUDA;
        attr_set = true;
    }
    kern<<<dim3(d2d_cdiv(D.d_h, 8), n_layers), NT, smem, st>>>((const TT *)x, T, D.d, D.d_h, D.n_experts, stage_w2, zero_words, args);
    D2D_LAUNCHED(1);
    return cudaGetLastError() == cudaSuccess ? D2D_OK : D2D_ERR_CUDA;
}

template <typename TT>
d2d_status launch_router(const d2d_layer_desc &D, int n, const SmallRouterArgs &a, const void *x, int T, int zero_words,
                         cudaStream_t st)
{
    switch (token_block(T)) {
    case 1: return launch_router_tb<TT, 1>(D, n, a, x, T, zero_words, st);
    case 2: return launch_router_tb<TT, 2>(D, n, a, x, T, zero_words, st);
    case 4: return launch_router_tb<TT, 4>(D, n, a, x, T, zero_words, st);
    default: return launch_router_tb<TT, 8>(D, n, a, x, T, zero_words, st);
    }
}

SmallSel make_sel(const d2d_routing *into, float tau)
{
    SmallSel sel = {};
    if (into) {
        sel.enabled = 1;
        sel.tau = tau;
        sel.mask = into->mask; sel.k = into->k; sel.counts = into->counts;
        sel.offsets = into->offsets; sel.perm = into->perm; sel.tok_off = into->tok_off;
        sel.tok_exp = into->tok_exp; sel.n_sel = into->n_sel; sel.status = into->status;
        sel.capacity = (long long)into->perm_capacity;
    }
    return sel;
}

}  // namespace

// ws: [ticket (256 bytes) | u: T*d_h floats]
size_t d2d_small_router_ws_bytes(const d2d_layer *L, int T) { return 256 + d2d_align_up((size_t)T * L->desc.d_h * 4, 256); }

bool d2d_small_router_supports(const d2d_layer_desc &D, int T)
{
    const size_t elem = D.dtype == D2D_F32 ? 4 : 2;
    return T >= 1 && T <= (D.dtype == D2D_BF16 ? d2d_decode_max_tokens(D) : 8) && D.d % 8 == 0 && D.d_h % 8 == 0 &&
           (size_t)(8 + MAX_TBLK) * D.d * elem + (size_t)T * D.d_h * 4 + (size_t)T * ((D.n_experts + 31) / 32) * 4 <= kSmemLimit;
}

d2d_status d2d_small_router(const d2d_layer *L, const void *x, int T, float *R, void *ws, cudaStream_t st,
                            const d2d_routing *select_into, float tau, int fused, float *zero, int zero_words)
{
    unsigned int *ticket = fused ? L->tickets : (unsigned int *)ws;
    float *u = (float *)((char *)ws + 256);
    if (!fused) D2D_CUDA_TRY(cudaMemsetAsync(ticket, 0, sizeof(unsigned int), st));
    SmallRouterArgs a = {};
    a.l[0] = {L->w_r1, L->b_r1, L->w_r2, L->b_r2, u, R, ticket, zero, make_sel(select_into, tau)};
    if (L->desc.dtype == D2D_F32) return launch_router<float>(L->desc, 1, a, x, T, zero_words, st);
    return launch_router<__nv_bfloat16>(L->desc, 1, a, x, T, zero_words, st);
}

// Decode batches of a layer group (layers of one shape reading the same tokens): ONE router launch (+ selection +
// metadata) and ONE expert launch for all layers.  Uses the layer-owned tickets; R[l], u[l] and y32[l] are scratch of the
// group's workspace; y is [n, T, d].
d2d_status d2d_small_group_fwd(const d2d_layer *const *layers, int n, const void *x, int T, float tau, const d2d_routing *routing,
                               float *const *R, float *const *u, float *const *y32, void *y, cudaStream_t st)
{
    if (n < 1 || n > D2D_MAX_GROUP) return D2D_ERR_INVALID_ARG;
    const d2d_layer_desc &D = layers[0]->desc;
    const size_t el = layers[0]->elem;
    SmallRouterArgs ra = {};
    SmallFfnArgs fa = {};
    for (int l = 0; l < n; ++l) {
        const d2d_layer *L = layers[l];
        ra.l[l] = {L->w_r1, L->b_r1, L->w_r2, L->b_r2, u[l], R[l], L->tickets, y32[l], make_sel(&routing[l], tau)};
        fa.l[l] = {L->w1, L->b1, L->w_gate, L->w2t, L->b2, routing[l].offsets, routing[l].perm, y32[l], L->tickets + 16,
                   (char *)y + (size_t)l * T * D.d * el, (long long)routing[l].perm_capacity};
    }
    d2d_status rc = D.dtype == D2D_F32 ? launch_router<float>(D, n, ra, x, T, T * D.d, st)
                                       : launch_router<__nv_bfloat16>(D, n, ra, x, T, T * D.d, st);
    if (rc != D2D_OK) return rc;
    return D.dtype == D2D_F32 ? launch_ffn_dtype<float>(D, n, fa, x, T, st) : launch_ffn_dtype<__nv_bfloat16>(D, n, fa, x, T, st);
}

// ws: [ticket (256 bytes) | y32: T*d floats]
size_t d2d_small_ffn_ws_bytes(const d2d_layer *L, int T) { return 256 + d2d_align_up((size_t)T * L->desc.d * 4, 256); }

bool d2d_small_ffn_supports(const d2d_layer_desc &D)
{
    return D.d % 8 == 0 && rows_per_pass(D, D.dtype == D2D_F32 ? 4 : 2) > 0;
}

d2d_status d2d_small_ffn(const d2d_layer *L, const void *x, int T, const d2d_routing *r, void *y, void *ws, cudaStream_t st,
                         int fused)
{
    unsigned int *ticket = fused ? L->tickets + 16 : (unsigned int *)ws;
    float *y32 = (float *)((char *)ws + 256);
    // the ticket and the float32 accumulator must start at zero
    if (!fused) D2D_CUDA_TRY(cudaMemsetAsync(ws, 0, 256 + (size_t)T * L->desc.d * 4, st));
    SmallFfnArgs a = {};
    a.l[0] = {L->w1, L->b1, L->w_gate, L->w2t, L->b2, r->offsets, r->perm, y32, ticket, y, (long long)r->perm_capacity};
    if (L->q_w1 && L->desc.d % 16 == 0) {                     // 8-bit expert weights: the kernel reads the codes
        a.l[0].w1 = L->q_w1; a.l[0].w_gate = L->q_wg; a.l[0].w2t = L->q_w2t;
        a.l[0].k1 = L->q_k1; a.l[0].kg = L->q_kg; a.l[0].k2 = L->q_k2;
    }
    if (L->desc.dtype == D2D_F32) return launch_ffn_dtype<float>(L->desc, 1, a, x, T, st);
    return launch_ffn_dtype<__nv_bfloat16>(L->desc, 1, a, x, T, st);
}
