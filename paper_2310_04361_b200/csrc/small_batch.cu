// Small-batch (decode) path: T <= 64 tokens.  Here the layer is bound by HBM traffic and by launch
// latency, not by arithmetic: every selected expert's weight slice is read exactly once, with
// 16-byte loads, by a CTA of its own, and the number of launches is kept to a minimum.
//
//   small_select_kernel   one CTA does the whole selection: row max, threshold, mask words, k,
//                         per-expert counts, offsets, token lists (and the token-major dual)
// The router and expert kernels of this path are in small_batch_ffn.cu.
#include "d2d_common.cuh"
#include "small_select.cuh"

namespace {

// ------------------------------------------------------------------------------------ selection

__global__ void __launch_bounds__(1024)
small_select_kernel(const float *__restrict__ R, int T, int E, int W, float tau,
                    uint32_t *__restrict__ mask, int32_t *__restrict__ k, int32_t *__restrict__ counts,
                    int32_t *__restrict__ offsets, int32_t *__restrict__ perm, int32_t *__restrict__ tok_off,
                    int32_t *__restrict__ tok_exp, int32_t *__restrict__ n_sel, int32_t *__restrict__ status,
                    long long capacity, int keep_status)
{
    extern __shared__ uint32_t smask[];          // [T][W]
    d2d_small::select_cta(R, T, E, W, tau, mask, k, counts, offsets, perm, tok_off, tok_exp, n_sel, status, capacity,
                          keep_status, smask);
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

