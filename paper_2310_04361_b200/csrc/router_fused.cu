// Fused router + dynamic-k mask for bf16 layers (Sec. 3.3 and Eq. 4): one kernel computes
//   u = relu(x W_r1^T + b_r1)            tcgen05 GEMM, 128 tokens x d_h, accumulator in TMEM
//   R = | u W_r2^T + b_r2 |              second tcgen05 GEMM whose A operand is u, written by the first
//                                        epilogue straight into shared memory in the swizzled K-major layout
//   m = max_i R[t,i], thr = tau * m (one fp32 RN multiply), mask words, k[t]     per-row epilogue on TMEM
// so the hidden activations never touch HBM, R is written once (the caller may want it) and the
// mask kernel's extra pass over R disappears.  One CTA per 128 tokens; 18 warps: TMA producer,
// MMA issuer, 16 epilogue warps (four per TMEM lane quadrant, each a quarter of the columns).
// All mbarrier waits are bounded (status D2D_ERR_TIMEOUT); every load is a plain per-CTA load.
#include <cuda.h>

#include "d2d_common.cuh"
#include "gemm_tc.cuh"
#include "tc_common.cuh"

namespace {

using d2d_tc::smem_u32; using d2d_tc::mbar_init; using d2d_tc::mbar_expect_tx; using d2d_tc::mbar_arrive;
using d2d_tc::tma_load_2d; using d2d_tc::smem_desc_sw128; using d2d_tc::instr_desc_bf16; using d2d_tc::umma_bf16;
using d2d_tc::umma_commit; using d2d_tc::tmem_ld16_issue; using d2d_tc::tmem_ld_wait;

constexpr int BM = 128, BK = 64, UMMA_K = 16;
constexpr int STAGES = 5;          // 5 x 32 KB of operands in flight: the first GEMM's main loop is bound by load latency
constexpr int NTHREADS = 64 + 512;       // TMA warp, MMA warp, 16 epilogue warps

// every barrier wait of this kernel: 4096 back-to-back polls, then one poll every 128 ns
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int32_t *status)
{
    return d2d_tc::mbar_wait<4096, 128>(bar, parity, status);
}
// 16 accumulator columns of this thread's TMEM lane, complete on return
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16])
{
    tmem_ld16_issue(taddr, r);
    tmem_ld_wait();
}

struct RouterLayerIO {
    float *R;              // [T, E] scores or NULL
    uint32_t *mask;        // [T, ceil(E/32)]
    int32_t *k;            // [T]
    int32_t *status;
};
struct RouterGroupIO {
    RouterLayerIO l[D2D_MAX_GROUP];
    uint32_t *mask_cat;    // merged mask [T, cat_words] or NULL
    int cat_words;
    int32_t *ksum;         // single layer only, or NULL: [0] running sum of k, [1] CTA exit ticket (both zero at launch and
                           // left at zero), [4] receives the total = number of selected (token, expert) pairs
};

// Shared memory (dynamic, 1024-byte aligned):
//   [ STAGES x (x tile 128x64 | W_r1 tile DH x 64) ]        first GEMM operand ring
//   [ u: DH/64 k-blocks x (128 rows x 128 B) ]              A operand of the second GEMM (written by epilogue 1)
//   W_r2 (DH/64 k-blocks x 256 rows x 128 B, the B operand of the second GEMM) reuses the first stages of the ring:
//   it is loaded as soon as the last k-blocks that used those stages have been consumed, under epilogue 1.
// TMEM: columns [0, DH) accumulator of u, columns [256, 256 + E_pad) accumulator of R (E <= 256).
// Several routers that read the same tokens (the Q, K and V projections of one attention layer) run as ONE grid:
// blockIdx.y picks the router.  Their weights are stacked (W_r1 [n*DH, d], b_r1 [n*DH], W_r2 [n*E, DH], b_r2 [n*E]);
// every router writes its own outputs and, when mask_cat is given, its mask words once more into a merged mask
// [T, cat_words] at word offset l * ceil(E/32) (the selection mask of the merged up projection).
template <int DH>
__global__ void __launch_bounds__(NTHREADS, 1)
router_fused_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w1,
                    const __grid_constant__ CUtensorMap tm_w2, const __nv_bfloat16 *__restrict__ b_r1_all,
                    const __nv_bfloat16 *__restrict__ b_r2_all, int T, int d, int E, int EN /* E rounded up to 16 */,
                    float tau, int do_mask, const __grid_constant__ RouterGroupIO io)
{
    const int layer = blockIdx.y;
    const __nv_bfloat16 *b_r1 = b_r1_all ? b_r1_all + layer * DH : nullptr;
    const __nv_bfloat16 *b_r2 = b_r2_all ? b_r2_all + layer * E : nullptr;
    float *__restrict__ R = io.l[layer].R;
    uint32_t *__restrict__ mask = io.l[layer].mask;
    int32_t *__restrict__ k = io.l[layer].k;
    int32_t *__restrict__ status = io.l[layer].status;
    constexpr int KB2 = DH / BK;                          // k-blocks of the second GEMM
    constexpr int A_BYTES = BM * BK * 2, B1_BYTES = DH * BK * 2;
    constexpr int STAGE_BYTES = A_BYTES + B1_BYTES;
    constexpr int U_BYTES = KB2 * BM * 128;
    constexpr int W2_KB_BYTES = 256 * 128;                // one k-block of W_r2 rows (box of 256 rows, zero filled past E)

    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *u_s = smem + (size_t)STAGES * STAGE_BYTES;
    uint8_t *w2_s = smem;                                  // aliases the first stages (see above)
    static_assert((size_t)KB2 * W2_KB_BYTES <= (size_t)STAGES * STAGE_BYTES, "W_r2 must fit in the operand ring");
    constexpr int W2_STAGES = (KB2 * W2_KB_BYTES + STAGE_BYTES - 1) / STAGE_BYTES;      // stages W_r2 overwrites
    __shared__ uint64_t bar_full[STAGES], bar_empty[STAGES], bar_w2, bar_acc1, bar_u_ready, bar_acc2;
    __shared__ uint32_t tmem_base_holder;
    __shared__ float b1_s[DH], b2_s[256];                  // biases as float32
    __shared__ float pmax_s[4 * BM];                       // per column-part row maxima
    __shared__ int pbad_s[4 * BM], pk_s[4 * BM];
    for (int i = threadIdx.x; i < DH; i += NTHREADS) b1_s[i] = b_r1 ? __bfloat162float(b_r1[i]) : 0.0f;
    for (int i = threadIdx.x; i < 256; i += NTHREADS) b2_s[i] = (b_r2 && i < E) ? __bfloat162float(b_r2[i]) : 0.0f;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m0 = blockIdx.x * BM;
    const int nkb = (d + BK - 1) / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        mbar_init(smem_u32(&bar_w2), 1);
        mbar_init(smem_u32(&bar_acc1), 1);
        mbar_init(smem_u32(&bar_u_ready), 16);            // one arrival per epilogue warp
        mbar_init(smem_u32(&bar_acc2), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_holder)),
                     "r"(512u)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_holder;
    const uint32_t tmem_r = tmem_base + 256;
    // the expert up projection that follows on the stream may start its operand loads and MMAs on the SMs this
    // grid leaves idle (T / 128 CTAs); its epilogue waits for this kernel to complete before it reads the mask
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            bool ok = true;
            for (int kb = 0; kb < nkb && ok; ++kb) {
                const uint32_t s = kb % STAGES, round = kb / STAGES;
                ok = mbar_wait(smem_u32(&bar_empty[s]), (round & 1u) ^ 1u, status);
                if (!ok) break;
                const uint32_t full = smem_u32(&bar_full[s]);
                const uint32_t dst = smem_u32(smem + (size_t)s * STAGE_BYTES);
                mbar_expect_tx(full, (uint32_t)STAGE_BYTES);
                tma_load_2d(dst, &tm_x, kb * BK, m0, full);
                tma_load_2d(dst + A_BYTES, &tm_w1, kb * BK, layer * DH, full);
            }
            // W_r2 goes into stages 0 .. W2_STAGES-1 once the MMAs of the last k-block that used each of them have retired
            for (int s = 0; s < W2_STAGES && ok; ++s) {
                if (s < nkb) {
                    const int last = s + ((nkb - 1 - s) / STAGES) * STAGES;      // last k-block held by stage s
                    ok = mbar_wait(smem_u32(&bar_empty[s]), (uint32_t)(last / STAGES) & 1u, status);
                }
            }
            if (ok) {
                mbar_expect_tx(smem_u32(&bar_w2), (uint32_t)(KB2 * W2_KB_BYTES));
                for (int kb = 0; kb < KB2; ++kb)
                    tma_load_2d(smem_u32(w2_s + (size_t)kb * W2_KB_BYTES), &tm_w2, kb * BK, layer * E, smem_u32(&bar_w2));
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            bool ok = true;
            const uint32_t idesc1 = instr_desc_bf16(BM, DH);
            for (int kb = 0; kb < nkb && ok; ++kb) {
                const uint32_t s = kb % STAGES, round = kb / STAGES;
                ok = mbar_wait(smem_u32(&bar_full[s]), round & 1u, status);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t a_addr = smem_u32(smem + (size_t)s * STAGE_BYTES);
                const uint64_t da = smem_desc_sw128(a_addr), db = smem_desc_sw128(a_addr + A_BYTES);
#pragma unroll
                for (int q = 0; q < BK / UMMA_K; ++q) {
                    const uint64_t koff = (uint64_t)((q * UMMA_K * 2) >> 4);
                    umma_bf16(tmem_base, da + koff, db + koff, idesc1, (kb | q) != 0 ? 1u : 0u);
                }
                umma_commit(smem_u32(&bar_empty[s]));
            }
            umma_commit(smem_u32(&bar_acc1));              // u accumulator complete
            // second GEMM: wait for u (written to shared memory by the epilogue warps) and for W_r2
            ok = ok && mbar_wait(smem_u32(&bar_u_ready), 0, status) && mbar_wait(smem_u32(&bar_w2), 0, status);
            if (ok) {
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t idesc2 = instr_desc_bf16(BM, EN);
                for (int kb = 0; kb < KB2; ++kb) {
                    const uint64_t da = smem_desc_sw128(smem_u32(u_s + (size_t)kb * BM * 128));
                    const uint64_t db = smem_desc_sw128(smem_u32(w2_s + (size_t)kb * W2_KB_BYTES));
#pragma unroll
                    for (int q = 0; q < BK / UMMA_K; ++q) {
                        const uint64_t koff = (uint64_t)((q * UMMA_K * 2) >> 4);
                        umma_bf16(tmem_r, da + koff, db + koff, idesc2, (kb | q) != 0 ? 1u : 0u);
                    }
                }
            }
            umma_commit(smem_u32(&bar_acc2));
        }
    } else {
        // ------------------------------------------------------------------ 16 epilogue warps
        // warp -> TMEM lane quadrant (warp & 3) and one of four column parts; a thread owns one token row
        const int quad = warp & 3, part = (warp - 2) >> 2;
        const int r_local = quad * 32 + lane;
        const int row = m0 + r_local;
        const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
        int okw = 1;
        if (lane == 0) okw = mbar_wait(smem_u32(&bar_acc1), 0, status) ? 1 : 0;
        bool ok = __shfl_sync(0xffffffffu, okw, 0) != 0;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (ok) {
            // ---- epilogue 1: u = relu(acc + b_r1) -> bf16 -> swizzled K-major tile in shared memory
            constexpr int C1 = DH / 4;                     // columns of u per part
#pragma unroll
            for (int cc = 0; cc < C1; cc += 16) {
                const int c0 = part * C1 + cc;
                uint32_t acc[16];
                tmem_ld16(tmem_base + lane_base + (uint32_t)c0, acc);
                uint32_t pk[8];
#pragma unroll
                for (int j = 0; j < 16; j += 2) {
                    const __nv_bfloat162 v = __floats2bfloat162_rn(fmaxf(__uint_as_float(acc[j]) + b1_s[c0 + j], 0.0f),
                                                                   fmaxf(__uint_as_float(acc[j + 1]) + b1_s[c0 + j + 1], 0.0f));
                    pk[j >> 1] = *reinterpret_cast<const uint32_t *>(&v);
                }
                // 16 columns = two 16-byte chunks of this row inside k-block c0/64; chunk index XOR (row % 8)
                const int kb = c0 >> 6, chunk = (c0 & 63) >> 3;
                uint8_t *rowp = u_s + (size_t)kb * BM * 128 + (size_t)r_local * 128;
                *reinterpret_cast<uint4 *>(rowp + (((chunk) ^ (r_local & 7)) << 4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                *reinterpret_cast<uint4 *>(rowp + (((chunk + 1) ^ (r_local & 7)) << 4)) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
            }
            // make the generic-proxy writes visible to the tensor-core (async) proxy, then signal the MMA warp
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bar_u_ready));

            // ---- epilogue 2: R = |acc + b_r2|; part p owns mask words p and p + 4 (columns 32w .. 32w+31)
            if (lane == 0) okw = mbar_wait(smem_u32(&bar_acc2), 0, status) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, okw, 0) != 0;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const int W = (E + 31) / 32;
            float v[2][32];
            float m = -INFINITY;
            bool bad = false;
            if (ok) {
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                    const int w = part + 4 * q;
                    if (w < W) {
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            const int c0 = w * 32 + h * 16;
                            if (c0 < EN) {
                                uint32_t acc[16];
                                tmem_ld16(tmem_r + lane_base + (uint32_t)c0, acc);
#pragma unroll
                                for (int j = 0; j < 16; ++j) {
                                    const int i = c0 + j;
                                    const float val = fabsf(__uint_as_float(acc[j]) + b2_s[i]);
                                    v[q][h * 16 + j] = val;
                                    if (i < E) {
                                        bad |= (__float_as_uint(val) & 0x7f800000u) == 0x7f800000u;
                                        m = val > m ? val : m;
                                    }
                                }
                                if (R && row < T) {
                                    float *o = R + (size_t)row * E + c0;
                                    if (c0 + 16 <= E && (E & 7) == 0 && (reinterpret_cast<uintptr_t>(R) & 31) == 0) {
                                        // 32-byte stores: a whole sector per lane and instruction
#pragma unroll
                                        for (int j = 0; j < 16; j += 8)
                                            asm volatile("st.global.v8.f32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(o + j),
                                                         "f"(v[q][h * 16 + j]), "f"(v[q][h * 16 + j + 1]), "f"(v[q][h * 16 + j + 2]),
                                                         "f"(v[q][h * 16 + j + 3]), "f"(v[q][h * 16 + j + 4]), "f"(v[q][h * 16 + j + 5]),
                                                         "f"(v[q][h * 16 + j + 6]), "f"(v[q][h * 16 + j + 7]) : "memory");
                                    } else if (c0 + 16 <= E && (E & 3) == 0) {
#pragma unroll
                                        for (int j = 0; j < 16; j += 4)
                                            *reinterpret_cast<float4 *>(o + j) = make_float4(v[q][h * 16 + j], v[q][h * 16 + j + 1],
                                                                                             v[q][h * 16 + j + 2], v[q][h * 16 + j + 3]);
                                    } else {
#pragma unroll
                                        for (int j = 0; j < 16; ++j)
                                            if (c0 + j < E) o[j] = v[q][h * 16 + j];
                                    }
                                }
                            } else {
#pragma unroll
                                for (int j = 0; j < 16; ++j) v[q][h * 16 + j] = 0.0f;
                            }
                        }
                    }
                }
            }
            if (do_mask) {
                // row maximum across the four column parts (and the non-finite flag), through shared memory
                pmax_s[part * BM + r_local] = m;
                pbad_s[part * BM + r_local] = bad ? 1 : 0;
                asm volatile("bar.sync 1, 512;" ::: "memory");           // the 16 epilogue warps only
                float mm = pmax_s[r_local];
                int anybad = pbad_s[r_local];
#pragma unroll
                for (int p = 1; p < 4; ++p) {
                    const float o = pmax_s[p * BM + r_local];
                    mm = o > mm ? o : mm;
                    anybad |= pbad_s[p * BM + r_local];
                }
                const float thr = __fmul_rn(tau, mm);
                int kt = 0;
                if (ok) {
#pragma unroll
                    for (int q = 0; q < 2; ++q) {
                        const int w = part + 4 * q;
                        if (w < W) {
                            uint32_t word = 0u;
#pragma unroll
                            for (int j = 0; j < 32; ++j) {
                                const int i = w * 32 + j;
                                if (i < E && (anybad || v[q][j] >= thr)) word |= 1u << j;
                            }
                            if (row < T) {
                                mask[(size_t)row * W + w] = word;
                                if (io.mask_cat) io.mask_cat[(size_t)row * io.cat_words + layer * W + w] = word;
                            }
                            kt += __popc(word);
                        }
                    }
                }
                pk_s[part * BM + r_local] = kt;
                asm volatile("bar.sync 1, 512;" ::: "memory");
                int k_row = 0;
                if (part == 0 && row < T) {
                    k_row = pk_s[r_local] + pk_s[BM + r_local] + pk_s[2 * BM + r_local] + pk_s[3 * BM + r_local];
                    k[row] = k_row;
                    if (anybad) atomicMax(status, (int32_t)D2D_ERR_NONFINITE);
                }
                if (io.ksum) {
                    // number of selected pairs of the whole batch, for the density-adaptive dispatch of the expert step
                    if (part == 0) {
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) k_row += __shfl_xor_sync(0xffffffffu, k_row, o);
                        if (lane == 0) atomicAdd(io.ksum, k_row);
                    }
                    asm volatile("bar.sync 1, 512;" ::: "memory");
                    if (warp == 2 && lane == 0) {
                        __threadfence();
                        if (atomicAdd(io.ksum + 1, 1) == (int)(gridDim.x * gridDim.y) - 1) {
                            __threadfence();
                            io.ksum[4] = atomicExch(io.ksum, 0);         // the CTA that finishes last publishes and resets
                            io.ksum[1] = 0;
                        }
                    }
                }
            }
        } else if (do_mask) {
            // keep the named barrier balanced when a bounded wait ran out
            asm volatile("bar.sync 1, 512;" ::: "memory");
            asm volatile("bar.sync 1, 512;" ::: "memory");
            if (io.ksum) asm volatile("bar.sync 1, 512;" ::: "memory");
        }
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

template <int DH>
d2d_status launch(const d2d_layer_desc &D, const d2d_router_weights &w, int n_layers, const void *x, int T, float tau, int do_mask,
                  const RouterGroupIO &io, cudaStream_t st)
{
    constexpr int STAGE_BYTES = BM * BK * 2 + DH * BK * 2;
    constexpr int KB2 = DH / BK;
    constexpr size_t SMEM = (size_t)STAGES * STAGE_BYTES + (size_t)KB2 * BM * 128 + 1024;
    CUtensorMap tx, tw1, tw2;
    if (!d2d_tc_make_map(&tx, x, T, D.d, BM) || !d2d_tc_make_map(&tw1, w.w_r1, D.d_h * n_layers, D.d, DH) ||
        !d2d_tc_make_map(&tw2, w.w_r2, D.n_experts * n_layers, D.d_h, 256))
        return D2D_ERR_CUDA;
    auto kern = router_fused_kernel<DH>;
    static bool attr_set[64] = {};                         // the attribute is per device
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return D2D_ERR_CUDA;
    if (!__atomic_load_n(&attr_set[dev], __ATOMIC_ACQUIRE)) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM) != cudaSuccess) return D2D_ERR_CUDA;
        __atomic_store_n(&attr_set[dev], true, __ATOMIC_RELEASE);
    }
    const int EN = (D.n_experts + 15) / 16 * 16;
    kern<<<dim3(d2d_cdiv(T, BM), n_layers), NTHREADS, SMEM, st>>>(tx, tw1, tw2, (const __nv_bfloat16 *)w.b_r1, (const __nv_bfloat16 *)w.b_r2,
                                                                 T, D.d, D.n_experts, EN, tau, do_mask, io);
    D2D_LAUNCHED(1);
    return cudaGetLastError() == cudaSuccess ? D2D_OK : D2D_ERR_CUDA;
}

}  // namespace

bool d2d_router_fused_supports(const d2d_layer_desc &D, int T)
{
    // d_h = 128 (the paper's router width) and E <= 256: operand ring, u and W_r2 then fit in shared memory together
    return D.dtype == D2D_BF16 && T > d2d_decode_max_tokens(D) && D.d_h == 128 && D.n_experts <= 256 && D.d % 8 == 0 && d2d_gemm_tc_available();
}

// R may be NULL when only the mask is wanted; mask / k / status are used when do_mask != 0.
d2d_status d2d_router_fused(const d2d_layer *L, const void *x, int T, float tau, int do_mask, float *R, uint32_t *mask,
                            int32_t *k, int32_t *status, cudaStream_t st, int32_t *ksum)
{
    RouterGroupIO io = {};
    io.l[0] = {R, mask, k, status};
    io.ksum = do_mask ? ksum : nullptr;
    const d2d_router_weights w = {L->w_r1, L->b_r1, L->w_r2, L->b_r2};
    return launch<128>(L->desc, w, 1, x, T, tau, do_mask, io, st);
}

// n routers of one shape with stacked weights, one grid; routing[l] receives mask, k and status of router l.
d2d_status d2d_router_fused_group(const d2d_layer_desc &D, const d2d_router_weights &w, int n_layers, const void *x, int T,
                                  float tau, const d2d_routing *routing, uint32_t *mask_cat, int cat_words, cudaStream_t st)
{
    if (n_layers < 1 || n_layers > D2D_MAX_GROUP) return D2D_ERR_INVALID_ARG;
    RouterGroupIO io = {};
    for (int l = 0; l < n_layers; ++l) io.l[l] = {nullptr, routing[l].mask, routing[l].k, routing[l].status};
    io.mask_cat = mask_cat;
    io.cat_words = cat_words;
    return launch<128>(D, w, n_layers, x, T, tau, 1, io, st);
}
