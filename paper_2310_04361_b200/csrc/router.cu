// router_fwd (Sec. 3.3): R = | W_r2 relu(W_r1 x + b_r1) + b_r2 |.
//
// Generic CUDA-core path: two launches of a shared-memory tiled kernel
// C[M,N] = epi(A[M,K] W[N,K]^T + b), float32 accumulation, hidden activations u kept
// in float32 in the workspace.  It covers every dtype and shape (fp32 layers must not
// go through reduced-precision tensor-core formats to stay within 1e-4).
#include "d2d_common.cuh"
#include "gemm_tc.cuh"

namespace {

constexpr int BM = 64, BN = 64, BK = 32, NT = 256;
enum { EPI_RELU = 0, EPI_ABS = 1 };

template <typename TA, typename TW, int EPI>
__global__ void __launch_bounds__(NT)
linear_epi_kernel(const TA *__restrict__ A, const TW *__restrict__ W, const TW *__restrict__ bias,
                  float *__restrict__ C, int M, int N, int K)
{
    __shared__ float As[BK][BM + 4];
    __shared__ float Ws[BK][BN + 4];
    const int tid = threadIdx.x;
    const int m0 = blockIdx.x * BM, n0 = blockIdx.y * BN;
    const int tx = tid % 16, ty = tid / 16;   // thread computes rows ty*4.., cols tx*4..
    float acc[4][4] = {};

    for (int k0 = 0; k0 < K; k0 += BK) {
        // 64 rows x 32 k-values per operand, 256 threads: 8 values each
        for (int i = tid; i < BM * BK; i += NT) {
            const int r = i / BK, c = i % BK;
            const int gm = m0 + r, gk = k0 + c;
            As[c][r] = (gm < M && gk < K) ? d2d_to_float<TA>(A[(size_t)gm * K + gk]) : 0.0f;
            const int gn = n0 + r;
            Ws[c][r] = (gn < N && gk < K) ? d2d_to_float<TW>(W[(size_t)gn * K + gk]) : 0.0f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float a[4], w[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) w[j] = Ws[kk][tx * 4 + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], w[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int gm = m0 + ty * 4 + i;
        if (gm >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int gn = n0 + tx * 4 + j;
            if (gn >= N) continue;
            float v = acc[i][j] + (bias ? d2d_to_float<TW>(bias[gn]) : 0.0f);
            v = (EPI == EPI_RELU) ? fmaxf(v, 0.0f) : fabsf(v);
            C[(size_t)gm * N + gn] = v;
        }
    }
}

template <typename T>
d2d_status run_router(const d2d_layer *L, const void *x, int Tn, float *R, float *u, cudaStream_t st)
{
    const int d = L->desc.d, d_h = L->desc.d_h, E = L->desc.n_experts;
    dim3 g1(d2d_cdiv(Tn, BM), d2d_cdiv(d_h, BN));
    linear_epi_kernel<T, T, EPI_RELU><<<g1, NT, 0, st>>>((const T *)x, (const T *)L->w_r1, (const T *)L->b_r1, u, Tn, d_h, d);
    dim3 g2(d2d_cdiv(Tn, BM), d2d_cdiv(E, BN));
    linear_epi_kernel<float, T, EPI_ABS><<<g2, NT, 0, st>>>(u, (const T *)L->w_r2, (const T *)L->b_r2, R, Tn, E, d_h);
    D2D_LAUNCHED(2);
    return cudaGetLastError() == cudaSuccess ? D2D_OK : D2D_ERR_CUDA;
}

}  // namespace

d2d_status d2d_launch_router(const d2d_layer *L, const void *x, int T, float *R, float *u_ws, cudaStream_t st)
{
    if (T == 0) return D2D_OK;
    // u_ws points at [256-byte ticket area | T*d_h floats]
    float *u = (float *)((char *)u_ws + 256);
    if (d2d_small_router_supports(L->desc, T)) return d2d_small_router(L, x, T, R, u_ws, st);
    if (d2d_router_fused_supports(L->desc, T)) return d2d_router_fused(L, x, T, 0.0f, 0, R, nullptr, nullptr, nullptr, st);
    if (L->desc.dtype == D2D_F32) return run_router<float>(L, x, T, R, u, st);
    if (d2d_gemm_tc_available()) {
        // bf16 layers: both router layers are dense contractions on the tensor cores; the hidden
        // activations u are kept in bf16 (they are the A operand of the second GEMM)
        const d2d_layer_desc &D = L->desc;
        d2d_gemm_args l1 = {};
        l1.a = x; l1.b = L->w_r1; l1.bias = L->b_r1; l1.out = u;
        l1.M = T; l1.N = D.d_h; l1.K = D.d; l1.epilogue = D2D_EPI_RELU_BF16;
        d2d_status rc = d2d_gemm_tc(l1, st);
        if (rc != D2D_OK) return rc;
        d2d_gemm_args l2 = {};
        l2.a = u; l2.b = L->w_r2; l2.bias = L->b_r2; l2.out = R;
        l2.M = T; l2.N = D.n_experts; l2.K = D.d_h; l2.epilogue = D2D_EPI_ABS_F32;
        return d2d_gemm_tc(l2, st);
    }
    return run_router<__nv_bfloat16>(L, x, T, R, u, st);
}
