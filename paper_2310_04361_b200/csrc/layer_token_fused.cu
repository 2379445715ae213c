// The whole layer of a SMALL problem in one launch (Sec. 3.2-3.4): router, dynamic-k rule, kept experts, combine.
//
// One CTA per token.  The token row sits in shared memory as float32; the warps compute the router's hidden units
// (a sub-warp per unit: a d-long dot product reduced by shuffles, bias + ReLU), then the expert scores (a sub-warp per
// expert, absolute value, Sec. 3.3), warp 0 takes the row maximum, the threshold tau * max as ONE float32 product and
// the mask words (Eq. 4), and the CTA then runs the token's kept experts: all their hidden neurons in one pass (a
// sub-warp per neuron), then the down projection with the neurons split over thread groups; a fixed summation order, no
// atomics, y written once with b2 added once.  Loops over weights are unrolled so that their loads are in flight
// together: at this size the kernel's time is a chain of memory latencies, not arithmetic.  When the caller wants
// the per-expert lists (Listing 1), the CTA that finishes last (a ticket) builds them from the mask words of all
// tokens with the single-CTA selection routine, so that no further launch follows.
//
// This is the path of float32 layers whose whole forward pass is a few MFLOP: there the chain of separate router,
// selection and expert kernels (eight launches) is nothing but launch latency.  Arithmetic is exact float32 FMA.
#include "d2d_common.cuh"
#include "small_select.cuh"

namespace {

constexpr int NT = 256;
constexpr int NWARP = NT / 32;
constexpr int MAX_H = 2048;         // hidden neurons of one token's kept experts staged in shared memory: d_ff <= MAX_H
constexpr int MAX_COLS = 4;         // output columns per thread: d <= NT * MAX_COLS

struct FusedArgs {
    const void *x, *w_r1, *b_r1, *w_r2, *b_r2, *w1, *b1, *w_gate, *w2t, *b2;
    void *y;
    float *R_out;                   // [T, E] or NULL
    d2d_routing r;                  // mask, k, status required; lists optional as a set
    unsigned int *ticket;           // zero at launch, left at zero
    int T, d, d_h, d_ff, E, s, W, lists;
    float tau;
};

// Lanes that share one weight row of `len` elements (8 elements per lane and step): a power of two, at most a warp.
// Short rows leave room for several rows per warp at a time, which shortens the chain of dependent memory round trips.
__device__ __forceinline__ int lanes_per_row(int len)
{
    int l = 1;
    while (l < 32 && l * 8 < len) l <<= 1;
    return l;
}

// dot(row, vec) for the sub-warp of `lpr` lanes this lane belongs to (every lane of the warp must call it)
template <typename T>
__device__ __forceinline__ float subwarp_dot(const T *row, const float *vec, int len, int lpr, int sl, bool valid)
{
    float v = 0.0f;
    if (valid)
        for (int c = sl * 8; c < len; c += lpr * 8) {
            float wv[8];
            d2d_load8(row + c, wv);
#pragma unroll
            for (int i = 0; i < 8; ++i) v = fmaf(wv[i], vec[c + i], v);
        }
    for (int o = lpr >> 1; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

template <typename T, int ACT, bool GATED>
__global__ void __launch_bounds__(NT)
layer_token_fused_kernel(const FusedArgs a)
{
    extern __shared__ float smem[];
    float *xs = smem;                                   // [d]
    float *us = xs + a.d;                               // [d_h]
    float *Rs = us + a.d_h;                             // [E]
    float *hs = Rs + a.E;                               // [d_ff] hidden activations of the kept experts, [groups * d] partial sums
    int *kept = reinterpret_cast<int *>(hs + max(a.d_ff, NT * MAX_COLS));     // [E] kept experts of this token, ascending
    uint32_t *words = reinterpret_cast<uint32_t *>(kept + a.E);               // [W] this token's mask words
    uint32_t *smask = words + a.W;                      // [T * W] all tokens' words (last CTA, lists only)
    __shared__ int n_kept;
    __shared__ int is_last;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int t = blockIdx.x, d = a.d, s = a.s;
    const T *x = (const T *)a.x;

    for (int c = tid; c < d; c += NT) xs[c] = d2d_to_float<T>(x[(size_t)t * d + c]);
    __syncthreads();
    // ---- router hidden layer: u = ReLU(W_r1 x + b_r1)
    {
        const int lpr = lanes_per_row(d), rpw = 32 / lpr, sub = lane / lpr, sl = lane % lpr;
#pragma unroll 2
        for (int j0 = warp * rpw; j0 < a.d_h; j0 += NWARP * rpw) {
            const int j = j0 + sub;
            const bool valid = j < a.d_h;
            const float v = subwarp_dot((const T *)a.w_r1 + (size_t)(valid ? j : 0) * d, xs, d, lpr, sl, valid);
            if (valid && sl == 0) us[j] = fmaxf(v + (a.b_r1 ? d2d_to_float<T>(((const T *)a.b_r1)[j]) : 0.0f), 0.0f);
        }
    }
    __syncthreads();
    // ---- router output layer: R = |W_r2 u + b_r2|
    {
        const int lpr = lanes_per_row(a.d_h), rpw = 32 / lpr, sub = lane / lpr, sl = lane % lpr;
#pragma unroll 2
        for (int e0 = warp * rpw; e0 < a.E; e0 += NWARP * rpw) {
            const int e = e0 + sub;
            const bool valid = e < a.E;
            const float v = subwarp_dot((const T *)a.w_r2 + (size_t)(valid ? e : 0) * a.d_h, us, a.d_h, lpr, sl, valid);
            if (valid && sl == 0) Rs[e] = fabsf(v + (a.b_r2 ? d2d_to_float<T>(((const T *)a.b_r2)[e]) : 0.0f));
        }
    }
    __syncthreads();
    // ---- dynamic-k rule (Eq. 4): keep expert i iff R_i >= tau * max_j R_j, the product rounded once to float32
    if (warp == 0) {
        float m = -INFINITY;
        bool bad = false;
        for (int i = lane; i < a.E; i += 32) {
            const float v = Rs[i];
            bad |= !d2d_small::finite_f32(v);
            m = v > m ? v : m;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float other = __shfl_xor_sync(0xffffffffu, m, o);
            m = other > m ? other : m;
        }
        bad = __any_sync(0xffffffffu, bad);
        const float thr = __fmul_rn(a.tau, m);
        int kt = 0;
        for (int w = 0; w < a.W; ++w) {
            const int i = w * 32 + lane;
            const bool keep = i < a.E && (bad || Rs[i] >= thr);
            const uint32_t word = __ballot_sync(0xffffffffu, keep);
            if (lane == 0) {
                words[w] = word;
                a.r.mask[(size_t)t * a.W + w] = word;
            }
            kt += __popc(word);
        }
        int pos = 0;
        for (int w = 0; w < a.W; ++w) {                        // the kept experts in ascending order
            const uint32_t word = words[w];
            if ((word >> lane) & 1u) kept[pos + __popc(word & ((1u << lane) - 1u))] = w * 32 + lane;
            pos += __popc(word);
        }
        if (lane == 0) {
            a.r.k[t] = kt;
            n_kept = kt;
            if (bad) atomicMax(a.r.status, (int32_t)D2D_ERR_NONFINITE);
        }
    } else if (a.R_out) {
        for (int i = tid - 32; i < a.E; i += NT - 32) a.R_out[(size_t)t * a.E + i] = Rs[i];
    }
    __syncthreads();
    // ---- kept experts, up projection + activation: all hidden neurons of all kept experts in one pass
    const int n_hidden = n_kept * s;
    {
        const int lpr = lanes_per_row(d), rpw = 32 / lpr, sub = lane / lpr, sl = lane % lpr;
#pragma unroll 2
        for (int i0 = warp * rpw; i0 < n_hidden; i0 += NWARP * rpw) {
            const int idx = i0 + sub;
            const bool valid = idx < n_hidden;
            const size_t n = valid ? (size_t)kept[idx / s] * s + idx % s : 0;
            float up = subwarp_dot((const T *)a.w1 + n * d, xs, d, lpr, sl, valid);
            float gate = 0.0f;
            if (GATED) gate = subwarp_dot((const T *)a.w_gate + n * d, xs, d, lpr, sl, valid);
            if (valid && sl == 0) {
                if (a.b1) up += d2d_to_float<T>(((const T *)a.b1)[n]);
                hs[idx] = GATED ? d2d_activate<ACT>(gate) * up : d2d_activate<ACT>(up);
            }
        }
    }
    __syncthreads();
    // ---- down projection: a thread owns output columns; when d is smaller than the CTA the hidden neurons are split
    // over NT / d thread groups whose partial sums meet in shared memory.  Fixed order: deterministic.
    const int groups = d < NT ? NT / d : 1;
    const int grp = d < NT ? tid / d : 0, col0 = d < NT ? tid % d : tid;
    float acc[MAX_COLS];
#pragma unroll
    for (int i = 0; i < MAX_COLS; ++i) acc[i] = 0.0f;
    if (grp < groups) {
#pragma unroll 8
        for (int idx = grp; idx < n_hidden; idx += groups) {
            const float hv = hs[idx];
            const T *row = (const T *)a.w2t + ((size_t)kept[idx / s] * s + idx % s) * d;
#pragma unroll
            for (int i = 0; i < MAX_COLS; ++i) {
                const int c = col0 + NT * i;
                if (c < d) acc[i] = fmaf(hv, d2d_to_float<T>(__ldg(row + c)), acc[i]);
            }
        }
    }
    if (groups > 1) {
        __syncthreads();                                       // every reader of hs is done: reuse it for the partial sums
        if (grp < groups) hs[grp * d + col0] = acc[0];
        __syncthreads();
        if (tid < d) {
            float v = a.b2 ? d2d_to_float<T>(((const T *)a.b2)[tid]) : 0.0f;
            for (int q = 0; q < groups; ++q) v += hs[q * d + tid];
            ((T *)a.y)[(size_t)t * d + tid] = d2d_from_float<T>(v);
        }
    } else {
#pragma unroll
        for (int i = 0; i < MAX_COLS; ++i) {
            const int c = tid + NT * i;
            if (c < d) ((T *)a.y)[(size_t)t * d + c] = d2d_from_float<T>(acc[i] + (a.b2 ? d2d_to_float<T>(((const T *)a.b2)[c]) : 0.0f));
        }
    }
    if (!a.lists) return;
    // ---- per-expert lists: the CTA that finishes last builds them from everybody's mask words
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const unsigned int done = atomicAdd(a.ticket, 1u);
        is_last = done == gridDim.x - 1;
        if (is_last) *a.ticket = 0u;
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    d2d_small::select_cta(nullptr, a.T, a.E, a.W, a.tau, a.r.mask, a.r.k, a.r.counts, a.r.offsets, a.r.perm, a.r.tok_off, a.r.tok_exp,
                          a.r.n_sel, a.r.status, a.r.perm_capacity, 1, smask);
}

template <typename T, int ACT>
d2d_status launch_act(const FusedArgs &a, bool gated, size_t smem, cudaStream_t st)
{
    if (gated)
        layer_token_fused_kernel<T, ACT, true><<<a.T, NT, smem, st>>>(a);
    else
        layer_token_fused_kernel<T, ACT, false><<<a.T, NT, smem, st>>>(a);
    D2D_LAUNCHED(1);
    return cudaGetLastError() == cudaSuccess ? D2D_OK : D2D_ERR_CUDA;
}

}  // namespace

static size_t fused_smem_bytes(const d2d_layer_desc &D, int T, bool lists)
{
    const int W = (D.n_experts + 31) / 32;
    const int h = D.d_ff > NT * MAX_COLS ? D.d_ff : NT * MAX_COLS;
    return (size_t)(D.d + D.d_h + D.n_experts + h + D.n_experts + W) * 4 + (lists ? (size_t)T * W * 4 : 0);
}

// Small float32 problems only: the router's weights are read once per token out of L2 here, which is fine for a few
// hundred KB and wasteful beyond.
bool d2d_layer_token_fused_supports(const d2d_layer_desc &D, int T, bool lists)
{
    const int W = (D.n_experts + 31) / 32;
    if (D.dtype != D2D_F32 || T < 1 || D.d > NT * MAX_COLS || D.d_ff > MAX_H || D.d % 8 || D.d_h % 8) return false;
    if ((size_t)D.d * D.d_h + (size_t)D.d_h * D.n_experts > 65536) return false;
    if (lists && (T > d2d_small::MAX_T || (size_t)T * W * 4 > 24 * 1024)) return false;
    return fused_smem_bytes(D, T, lists) <= 44 * 1024;
}

d2d_status d2d_layer_token_fused(const d2d_layer *L, const void *x, int T, float tau, void *y, float *R_out, const d2d_routing *r,
                                 bool lists, unsigned int *ticket, cudaStream_t st)
{
    const d2d_layer_desc &D = L->desc;
    FusedArgs a = {};
    a.x = x; a.w_r1 = L->w_r1; a.b_r1 = L->b_r1; a.w_r2 = L->w_r2; a.b_r2 = L->b_r2;
    a.w1 = L->w1; a.b1 = L->b1; a.w_gate = L->w_gate; a.w2t = L->w2t; a.b2 = L->b2;
    a.y = y; a.R_out = R_out; a.r = *r; a.ticket = ticket;
    a.T = T; a.d = D.d; a.d_h = D.d_h; a.d_ff = D.d_ff; a.E = D.n_experts; a.s = D.expert_size; a.W = (D.n_experts + 31) / 32; a.lists = lists ? 1 : 0;
    a.tau = tau;
    const size_t smem = fused_smem_bytes(D, T, lists);
    switch (D.act) {
    case D2D_ACT_RELU: return launch_act<float, D2D_ACT_RELU>(a, D.gated != 0, smem, st);
    case D2D_ACT_GELU_ERF: return launch_act<float, D2D_ACT_GELU_ERF>(a, D.gated != 0, smem, st);
    case D2D_ACT_GELU_TANH: return launch_act<float, D2D_ACT_GELU_TANH>(a, D.gated != 0, smem, st);
    case D2D_ACT_SILU: return launch_act<float, D2D_ACT_SILU>(a, D.gated != 0, smem, st);
    }
    return D2D_ERR_INVALID_ARG;
}
