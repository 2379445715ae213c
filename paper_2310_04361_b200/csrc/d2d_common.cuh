// Shared declarations of the CUDA translation units behind include/d2d.h.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "d2d.h"

// Packed, library-owned copy of one layer's parameters.
struct d2d_layer {
    d2d_layer_desc desc;
    size_t elem;            // bytes per element of desc.dtype
    int sm_count;
    // router
    void *w_r1, *b_r1, *w_r2, *b_r2;
    // experts: w1 / w_gate as given ([d_ff, d], an expert = s contiguous rows),
    // w2t = W2 transposed to [d_ff, d] so that an expert's slice is s contiguous rows too
    void *w1, *b1, *w_gate, *w2t, *b2;
    void *w2;               // W2 as given ([d, d_ff]): the K-major B operand of the dense down projection
    void *w1g;              // gated bf16 layers: W1 and W_gate interleaved in blocks of 128 rows (see d2d_gemm_args::b_cat)
    void *slab;             // one allocation backing all of the above
    size_t slab_bytes;
    // side stream + events: the per-expert metadata (counts, offsets, token lists) is built beside the
    // expert GEMMs, which do not read it
    cudaStream_t side_stream;
    cudaEvent_t ev_fork, ev_join;
    cudaEvent_t ev_fill_fork, ev_fill_join;      // zero fill of H beside the gathered up projection (side stream)
    // 8-bit expert weights (d2d_layer_create_fp8): e4m3 codes [d_ff, d] of W1, W_gate and the transposed W2, one scale
    // exponent per expert and matrix; NULL for ordinary layers.  w1, w_gate, w2, w2t, w1g then hold the dequantised values.
    void *q_slab;
    uint8_t *q_w1, *q_wg, *q_w2t;
    int32_t *q_k1, *q_kg, *q_k2;
    // d2d_layer_fwd_host: copy-in and copy-out streams and per-chunk events, so that the host -> device copy of one
    // chunk of tokens, the layer on the previous chunk and the device -> host copy of the one before overlap
    static const int kHostChunks = 4;
    cudaStream_t copy_in, copy_out;
    cudaEvent_t ev_in[kHostChunks], ev_done[kHostChunks], ev_begin, ev_end;
    // layer-owned "last CTA" tickets of the decode kernels used by d2d_layer_fwd (zero at creation, reset by the kernel
    // that used them): word 0 decode router, word 16 decode experts, word 32 tile counter of the up projection, words
    // 40 / 41 sum of k and exit ticket of the fused router, word 44 the number of selected pairs the fused router
    // publishes for the density-adaptive dispatch of the expert step, word 52 exit ticket of the one-launch layer
    // kernel of small float32 problems.  Like the side stream, they make concurrent
    // d2d_layer_fwd calls on ONE layer object from several streams unsafe; use one layer object per stream for that.
    // A call that ended in D2D_ERR_TIMEOUT may leave them non-zero: d2d_layer_reset_counters clears them.
    unsigned int *tickets;
    // gathered expert path (moe_gather.cu): per-group sub-chunk counters + exit ticket (self-resetting like the tickets),
    // experts per group (0 = the shape cannot use the path), which path the expert step takes (d2d_expert_path) and
    // the density up to which the automatic choice takes the gathered path
    int *gather_ctr;
    int gather_ctr_words;
    int gather_group;
    int expert_path;
    double gather_rho_max;
    int fused_group;              // experts per group of the fused gathered kernel (0: shape not supported)
    double fused_rho_max;         // automatic choice: the fused kernel runs while n_sel <= fused_rho_max * T * E (0: never)
};

// Layers of one shape that read the same token rows (the Q, K and V projections of one attention layer) and run as
// one launch sequence; see d2d_group_fwd.
#define D2D_MAX_GROUP 4
struct d2d_router_weights {
    const void *w_r1, *b_r1, *w_r2, *b_r2;
};
struct d2d_group {
    int n;
    d2d_layer *layers[D2D_MAX_GROUP];        // not owned
    d2d_layer_desc desc;                     // the common shape
    int merged;                              // 1: the stacked copies below exist and the merged tensor-core path may be used
    // stacked copies: routers [n*d_h, d], [n*d_h], [n*E, d_h], [n*E]; W1 [n*d_ff, d], b1 [n*d_ff]; W2 [n*d, d_ff], b2 [n*d]
    void *w_r1, *b_r1, *w_r2, *b_r2, *w1, *b1, *w2, *b2;
    void *slab;
    int *up_counter;                         // tile counter of the merged up projection (inside the slab, self-resetting)
    cudaStream_t side_stream;
    cudaEvent_t ev_fork, ev_join;
};

#define D2D_CUDA_TRY(expr)                                   \
    do {                                                     \
        cudaError_t err__ = (expr);                          \
        if (err__ != cudaSuccess) return D2D_ERR_CUDA;       \
    } while (0)

// Host-side count of kernel launches (reported by d2d_launch_count()).
extern unsigned long long d2d_launch_counter;
#define D2D_LAUNCHED(n) __atomic_fetch_add(&d2d_launch_counter, (unsigned long long)(n), __ATOMIC_RELAXED)

// Largest batch served by the decode kernels (cp.async CUDA-core kernels, two launches per layer call); larger bf16
// batches take the tensor-core path.  4 by default, D2D_DECODE_MAX_TOKENS=n (0 .. 8) overrides it for tuning.
int d2d_decode_max_tokens(const d2d_layer_desc &D);

static inline size_t d2d_align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
static inline int d2d_cdiv(int a, int b) { return (a + b - 1) / b; }

// ---- launch wrappers implemented in the kernel files -------------------------------------

d2d_status d2d_launch_router(const d2d_layer *L, const void *x, int T, float *R, float *u_ws, cudaStream_t st);

size_t d2d_select_ws_bytes(int T, int E);
// R == nullptr: the mask is an input.  mask_ready != 0: mask, k and the status word were already written
// (fused router), only the per-expert metadata is built.
d2d_status d2d_launch_dynk_mask(const float *R, int T, int E, float tau, const d2d_routing *out, int32_t *ksum, cudaStream_t st);
d2d_status d2d_launch_select(const float *R, int T, int E, float tau, int topk, const d2d_routing *out,
                             void *ws, cudaStream_t st, int mask_ready = 0);

// up_counter: see launch_tc_experts (NULL unless the fused router was launched just before on `st`)
// n_sel: device word that holds the number of selected pairs when the expert kernels start (NULL: r->n_sel)
d2d_status d2d_launch_moe_ffn(const d2d_layer *L, const void *x, int T, const d2d_routing *r, void *y,
                              void *ws, size_t ws_bytes, cudaStream_t st, int *up_counter = nullptr, int small_fused = 0,
                              const int32_t *n_sel = nullptr);
size_t d2d_moe_ffn_ws_bytes(const d2d_layer *L, int T);

// layer_token_fused.cu: the whole layer of a small float32 problem in one launch (router, rule, experts, lists).
// ticket: a zeroed layer-owned word (left at zero).  The status word must be zero (or hold an earlier error) at launch.
bool d2d_layer_token_fused_supports(const d2d_layer_desc &D, int T, bool lists);
d2d_status d2d_layer_token_fused(const d2d_layer *L, const void *x, int T, float tau, void *y, float *R_out, const d2d_routing *r,
                                 bool lists, unsigned int *ticket, cudaStream_t st);

// small-batch (T <= 64) kernels
bool d2d_small_select_supports(int T, int E);
d2d_status d2d_small_select(const float *R, int T, int E, float tau, const d2d_routing *out, cudaStream_t st,
                            int mask_ready = 0);
bool d2d_router_fused_supports(const d2d_layer_desc &D, int T);
// ksum (optional, 8 device ints, words 0 and 1 zero at launch and left at zero): the kernel adds up k over all tokens
// and its last CTA publishes the total, the number of selected (token, expert) pairs, in ksum[4]
d2d_status d2d_router_fused(const d2d_layer *L, const void *x, int T, float tau, int do_mask, float *R, uint32_t *mask,
                            int32_t *k, int32_t *status, cudaStream_t st, int32_t *ksum = nullptr);
d2d_status d2d_router_fused_group(const d2d_layer_desc &D, const d2d_router_weights &w, int n_layers, const void *x, int T,
                                  float tau, const d2d_routing *routing, uint32_t *mask_cat, int cat_words, cudaStream_t st);
d2d_status d2d_small_group_fwd(const d2d_layer *const *layers, int n, const void *x, int T, float tau, const d2d_routing *routing,
                               float *const *R, float *const *u, float *const *y32, void *y, cudaStream_t st);
bool d2d_small_router_supports(const d2d_layer_desc &D, int T);
size_t d2d_small_router_ws_bytes(const d2d_layer *L, int T);
// select_into != NULL: the kernel's last CTA also performs the dynamic-k selection (threshold tau) and writes the routing
// fused != 0 (d2d_layer_fwd): the layer-owned ticket is used (no memset node) and the kernel also clears `zero_words`
// floats at `zero` (the experts' float32 accumulator), so that the expert kernel needs no memset either
d2d_status d2d_small_router(const d2d_layer *L, const void *x, int T, float *R, void *ws, cudaStream_t st,
                            const d2d_routing *select_into = nullptr, float tau = 0.0f, int fused = 0,
                            float *zero = nullptr, int zero_words = 0);
bool d2d_small_ffn_supports(const d2d_layer_desc &D);
size_t d2d_small_ffn_ws_bytes(const d2d_layer *L, int T);
// fused != 0: the accumulator in ws was cleared by the router kernel and the layer-owned ticket is used
d2d_status d2d_small_ffn(const d2d_layer *L, const void *x, int T, const d2d_routing *r, void *y, void *ws, cudaStream_t st,
                         int fused = 0);

d2d_status d2d_launch_transpose(const void *src, void *dst, int rows, int cols, size_t elem, cudaStream_t st);

// quant_fp8.cu: per-expert e4m3 codes + power-of-two scale exponents of n_experts slices of per_expert bf16 weights;
// the weights are replaced in place by their dequantised values (exactly bf16)
d2d_status d2d_quantize_experts_e4m3(void *w, uint8_t *codes, int32_t *exps, int n_experts, int per_expert, cudaStream_t st);

// ---- device helpers ------------------------------------------------------------------------

#ifdef __CUDACC__

template <typename T> __device__ __forceinline__ float d2d_to_float(T v);
template <> __device__ __forceinline__ float d2d_to_float<float>(float v) { return v; }
template <> __device__ __forceinline__ float d2d_to_float<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T> __device__ __forceinline__ T d2d_from_float(float v);
template <> __device__ __forceinline__ float d2d_from_float<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 d2d_from_float<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// Activation of the hidden neurons; evaluated in float32 with the accurate libdevice routines.
template <int ACT> __device__ __forceinline__ float d2d_activate(float z)
{
    if (ACT == D2D_ACT_RELU) return fmaxf(z, 0.0f);
    if (ACT == D2D_ACT_GELU_ERF) return 0.5f * z * (1.0f + erff(z * 0.70710678118654752f));
    if (ACT == D2D_ACT_GELU_TANH) {
        const float c = 0.79788456080286536f;  // sqrt(2/pi)
        return 0.5f * z * (1.0f + tanhf(c * (z + 0.044715f * z * z * z)));
    }
    return z / (1.0f + expf(-z));  // SiLU
}

__device__ __forceinline__ float d2d_warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// 8 consecutive elements starting at p (16-byte aligned for bf16, 32-byte for float) as floats.
__device__ __forceinline__ void d2d_load8(const float *p, float (&o)[8])
{
    const float4 a = __ldg(reinterpret_cast<const float4 *>(p));
    const float4 b = __ldg(reinterpret_cast<const float4 *>(p) + 1);
    o[0] = a.x; o[1] = a.y; o[2] = a.z; o[3] = a.w; o[4] = b.x; o[5] = b.y; o[6] = b.z; o[7] = b.w;
}
__device__ __forceinline__ void d2d_load8(const __nv_bfloat16 *p, float (&o)[8])
{
    const uint4 raw = __ldg(reinterpret_cast<const uint4 *>(p));
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        o[2 * i] = __uint_as_float(w[i] << 16);
        o[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}

#endif  // __CUDACC__
