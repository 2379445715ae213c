// Low-precision expert weights (App. C runs the expert kernels on narrower number formats; here the weights of the
// expert step, Sec. 3.2, are held as 8-bit floating point).
//
// An expert's slice of W1, W_gate or W2 (s rows of d elements in the packed copies, W2 in its transposed copy) becomes
// s * d codes in the e4m3 format (1 sign, 4 exponent, 3 mantissa bits, bias 7, no infinities, largest value 448) and
// ONE exponent k: weight = value(code) * 2^k, with the smallest k for which the slice's largest magnitude fits.  A
// power-of-two scale makes every dequantised weight exactly a bfloat16 value, so the layer keeps a bf16 copy of the
// dequantised weights for the tensor-core paths and the results of all paths agree; the decode kernels, which are
// bound by the bytes of the kept experts, read the codes (half the bytes).
//
// One CTA per expert and matrix: maximum of the slice, exponent, then every element is scaled, converted with the
// hardware's round-to-nearest-even saturating conversion, and written twice: the code, and its value back in place.
#include <cuda_fp8.h>

#include "d2d_common.cuh"

namespace {

__global__ void __launch_bounds__(256)
quantize_experts_e4m3_kernel(__nv_bfloat16 *__restrict__ w, uint8_t *__restrict__ codes, int32_t *__restrict__ exps, int per_expert)
{
    __shared__ float red[8];
    __shared__ int k_s;
    const int e = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __nv_bfloat16 *we = w + (size_t)e * per_expert;
    uint8_t *ce = codes + (size_t)e * per_expert;
    float m = 0.0f;
    for (int i = threadIdx.x; i < per_expert; i += 256) m = fmaxf(m, fabsf(__bfloat162float(we[i])));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (lane == 0) red[warp] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
        float amax = 0.0f;
        for (int i = 0; i < 8; ++i) amax = fmaxf(amax, red[i]);
        // smallest k with amax <= 448 * 2^k, by exact comparisons (448 = 1.75 * 2^8)
        int k = 0;
        if (amax > 0.0f) {
            k = ilogbf(amax) - 8;
            if (amax > ldexpf(448.0f, k)) ++k;
        }
        k_s = k;
        exps[e] = k;
    }
    __syncthreads();
    const int k = k_s;
    for (int i = threadIdx.x; i < per_expert; i += 256) {
        const float v = ldexpf(__bfloat162float(we[i]), -k);                     // exact: a power-of-two scale
        const __nv_fp8_storage_t c = __nv_cvt_float_to_fp8(v, __NV_SATFINITE, __NV_E4M3);
        const __half_raw h = __nv_cvt_fp8_to_halfraw(c, __NV_E4M3);
        ce[i] = (uint8_t)c;
        we[i] = __float2bfloat16_rn(ldexpf(__half2float(*reinterpret_cast<const __half *>(&h)), k));   // exact as well
    }
}

}  // namespace

// w: [n_experts * per_expert] bf16 in place (dequantised values on return); codes: same count of bytes; exps: [n_experts]
d2d_status d2d_quantize_experts_e4m3(void *w, uint8_t *codes, int32_t *exps, int n_experts, int per_expert, cudaStream_t st)
{
    quantize_experts_e4m3_kernel<<<n_experts, 256, 0, st>>>((__nv_bfloat16 *)w, codes, exps, per_expert);
    D2D_LAUNCHED(1);
    return cudaGetLastError() == cudaSuccess ? D2D_OK : D2D_ERR_CUDA;
}
