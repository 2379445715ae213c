// moe_ffn_fwd, token-major CUDA-core path (Sec. 3.2, 3.4; gated form App. G).
//
// One CTA per token.  The token row sits in shared memory as float32; for each kept expert
// the warps compute the expert's s hidden neurons (one warp per neuron: a d-long dot product
// read with 16-byte loads and reduced by shuffles, bias + activation fused), then every
// thread owns a fixed set of output columns and accumulates h_n * W2T[n, :] into registers
// across all kept experts.  y is written once (b2 added once); no atomics, no scratch, and
// a fixed summation order (experts ascending), so the result is deterministic.
//
// Weight traffic is one expert slice per (token, expert) pair, which is exactly the touched
// bytes when a handful of tokens is decoded; for large batches the grouped tensor-core path
// is the one to use (this kernel stays as the exact fp32 path and as a cross-check).
#include "d2d_common.cuh"

namespace {

constexpr int NT = 256;
constexpr int NWARP = NT / 32;
constexpr int MAX_S = 128;          // largest expert size this kernel stages in shared memory
constexpr int MAX_COLS = 16;        // output columns per thread: d <= NT * MAX_COLS

template <typename T, int ACT, bool GATED>
__global__ void __launch_bounds__(NT)
moe_ffn_token_kernel(const T *__restrict__ x, int Tn, int d, int E, int s, int W,
                     const T *__restrict__ w1, const T *__restrict__ b1, const T *__restrict__ w_gate,
                     const T *__restrict__ w2t, const T *__restrict__ b2,
                     const uint32_t *__restrict__ mask, T *__restrict__ y)
{
    extern __shared__ float smem[];
    float *xs = smem;              // [d]
    float *hs = smem + d;          // [2][MAX_S] double-buffered hidden values
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    for (int t = blockIdx.x; t < Tn; t += gridDim.x) {
        __syncthreads();           // previous token's readers of xs / hs are done
        for (int c = tid; c < d; c += NT) xs[c] = d2d_to_float<T>(x[(size_t)t * d + c]);
        float acc[MAX_COLS];
#pragma unroll
        for (int i = 0; i < MAX_COLS; ++i) acc[i] = 0.0f;
        __syncthreads();

        int buf = 0;
        for (int w = 0; w < W; ++w) {
            uint32_t word = __ldg(mask + (size_t)t * W + w);
            while (word) {
                const int e = w * 32 + __ffs(word) - 1;
                word &= word - 1;
                float *h = hs + buf * MAX_S;
                // ---- up projection + activation: one warp per neuron
                for (int nl = warp; nl < s; nl += NWARP) {
                    const size_t n = (size_t)e * s + nl;
                    const T *wrow = w1 + n * d;
                    const T *grow = GATED ? w_gate + n * d : nullptr;
                    float up = 0.0f, gate = 0.0f;
                    for (int c = lane * 8; c < d; c += 256) {
                        float wv[8];
                        d2d_load8(wrow + c, wv);
#pragma unroll
                        for (int i = 0; i < 8; ++i) up = fmaf(wv[i], xs[c + i], up);
                        if (GATED) {
                            d2d_load8(grow + c, wv);
#pragma unroll
                            for (int i = 0; i < 8; ++i) gate = fmaf(wv[i], xs[c + i], gate);
                        }
                    }
                    up = d2d_warp_sum(up);
                    if (GATED) gate = d2d_warp_sum(gate);
                    if (lane == 0) {
                        if (b1) up += d2d_to_float<T>(b1[n]);
                        h[nl] = GATED ? d2d_activate<ACT>(gate) * up : d2d_activate<ACT>(up);
                    }
                }
                __syncthreads();
                // ---- down projection: thread owns columns tid + NT*i
                for (int nl = 0; nl < s; ++nl) {
                    const float hv = h[nl];
                    const T *row = w2t + ((size_t)e * s + nl) * d;
#pragma unroll
                    for (int i = 0; i < MAX_COLS; ++i) {
                        const int c = tid + NT * i;
                        if (c < d) acc[i] = fmaf(hv, d2d_to_float<T>(__ldg(row + c)), acc[i]);
                    }
                }
                buf ^= 1;          // the next expert writes the other buffer: one barrier per expert
            }
        }
#pragma unroll
        for (int i = 0; i < MAX_COLS; ++i) {
            const int c = tid + NT * i;
            if (c < d) {
                const float bias = b2 ? d2d_to_float<T>(b2[c]) : 0.0f;
                y[(size_t)t * d + c] = d2d_from_float<T>(acc[i] + bias);
            }
        }
    }
}

template <typename T, int ACT>
d2d_status launch_act(const d2d_layer *L, const void *x, int Tn, const d2d_routing *r, void *y, cudaStream_t st)
{
    const d2d_layer_desc &D = L->desc;
    const int W = (D.n_experts + 31) / 32;
    const size_t smem = sizeof(float) * ((size_t)D.d + 2 * MAX_S);
    const int grid = Tn;
    if (D.gated)
        moe_ffn_token_kernel<T, ACT, true><<<grid, NT, smem, st>>>(
            (const T *)x, Tn, D.d, D.n_experts, D.expert_size, W, (const T *)L->w1, (const T *)L->b1,
            (const T *)L->w_gate, (const T *)L->w2t, (const T *)L->b2, r->mask, (T *)y);
    else
        moe_ffn_token_kernel<T, ACT, false><<<grid, NT, smem, st>>>(
            (const T *)x, Tn, D.d, D.n_experts, D.expert_size, W, (const T *)L->w1, (const T *)L->b1,
            nullptr, (const T *)L->w2t, (const T *)L->b2, r->mask, (T *)y);
    D2D_LAUNCHED(1);
    return cudaGetLastError() == cudaSuccess ? D2D_OK : D2D_ERR_CUDA;
}

template <typename T>
d2d_status launch_dtype(const d2d_layer *L, const void *x, int Tn, const d2d_routing *r, void *y, cudaStream_t st)
{
    switch (L->desc.act) {
    case D2D_ACT_RELU: return launch_act<T, D2D_ACT_RELU>(L, x, Tn, r, y, st);
    case D2D_ACT_GELU_ERF: return launch_act<T, D2D_ACT_GELU_ERF>(L, x, Tn, r, y, st);
    case D2D_ACT_GELU_TANH: return launch_act<T, D2D_ACT_GELU_TANH>(L, x, Tn, r, y, st);
    case D2D_ACT_SILU: return launch_act<T, D2D_ACT_SILU>(L, x, Tn, r, y, st);
    }
    return D2D_ERR_INVALID_ARG;
}

// W2 [rows=d, cols=d_ff] -> W2T [d_ff, d], 32x32 shared-memory tiles.
template <typename T>
__global__ void transpose_kernel(const T *__restrict__ src, T *__restrict__ dst, int rows, int cols)
{
    __shared__ T tile[32][33];
    const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
    for (int i = threadIdx.y; i < 32; i += blockDim.y) {
        const int r = r0 + i, c = c0 + threadIdx.x;
        if (r < rows && c < cols) tile[i][threadIdx.x] = src[(size_t)r * cols + c];
    }
    __syncthreads();
    for (int i = threadIdx.y; i < 32; i += blockDim.y) {
        const int c = c0 + i, r = r0 + threadIdx.x;
        if (r < rows && c < cols) dst[(size_t)c * rows + r] = tile[threadIdx.x][i];
    }
}

}  // namespace

bool d2d_token_path_supports(const d2d_layer_desc &D)
{
    return D.expert_size <= MAX_S && D.d <= NT * MAX_COLS && D.d % 8 == 0;
}

d2d_status d2d_launch_moe_ffn_token(const d2d_layer *L, const void *x, int T, const d2d_routing *r, void *y,
                                    cudaStream_t st)
{
    if (T == 0) return D2D_OK;
    if (!d2d_token_path_supports(L->desc)) return D2D_ERR_UNSUPPORTED;
    if (L->desc.dtype == D2D_F32) return launch_dtype<float>(L, x, T, r, y, st);
    return launch_dtype<__nv_bfloat16>(L, x, T, r, y, st);
}

d2d_status d2d_launch_transpose(const void *src, void *dst, int rows, int cols, size_t elem, cudaStream_t st)
{
    dim3 grid(d2d_cdiv(cols, 32), d2d_cdiv(rows, 32)), block(32, 8);
    if (elem == 4)
        transpose_kernel<float><<<grid, block, 0, st>>>((const float *)src, (float *)dst, rows, cols);
    else
        transpose_kernel<__nv_bfloat16><<<grid, block, 0, st>>>((const __nv_bfloat16 *)src, (__nv_bfloat16 *)dst, rows, cols);
    return cudaGetLastError() == cudaSuccess ? D2D_OK : D2D_ERR_CUDA;
}
