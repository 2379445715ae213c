// bf16 GEMM C[M,N] = epilogue(A[M,K] B[N,K]^T) on the 5th-generation tensor cores of sm_100a.
//
//   warp 0   TMA producer: cp.async.bulk.tensor tiles of A (128 x 64) and B (BN x 64), 128-byte
//            swizzled, into a ring of shared-memory stages guarded by full/empty mbarriers
//   warp 1   allocates TMEM and issues tcgen05.mma (one thread), fp32 accumulator in TMEM;
//            tcgen05.commit releases a stage when the MMAs that read it have retired
//   warps 2-5  epilogue: tcgen05.ld the accumulator (one row per thread), bias / activation /
//            selection mask, vectorised stores
//
// Every mbarrier wait is bounded: when the limit runs out the role records D2D_ERR_TIMEOUT in the
// status word and leaves its loop, all roles meet at the final barrier, TMEM is freed and the
// kernel returns (no trap, no endless spin).  No multicast loads are used.
#include "gemm_tc.cuh"

namespace {

constexpr int BM = 128;          // rows of A per CTA = TMEM lanes
constexpr int BK = 64;           // 64 bf16 = one 128-byte swizzle row
constexpr int UMMA_K = 16;
constexpr int NTHREADS = 192;
constexpr uint32_t WAIT_LIMIT = 1u << 22;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bounded wait for the phase with the given parity; false (and status set) when the limit runs out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int32_t *status)
{
    for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(bar), "r"(parity)
            : "memory");
        if (done) return true;
        if (it > 32) __nanosleep(64);
    }
    if (status) atomicMax(status, (int32_t)D2D_ERR_TIMEOUT);
    return false;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int c0, int c1, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar)
        : "memory");
}

// K-major operand tile whose rows are 128 bytes, 128-byte swizzle: 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3fffu);
    d |= (uint64_t)1 << 16;                 // leading byte offset (not used by swizzled K-major layouts)
    d |= (uint64_t)(1024 >> 4) << 32;       // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                 // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                 // 128-byte swizzle
    return d;
}

__device__ __forceinline__ uint32_t instr_desc_bf16(int m, int n)
{
    return (1u << 4)                        // fp32 accumulator
           | (1u << 7) | (1u << 10)         // A and B are bf16
           | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);   // both operands K-major
}

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

struct EpiParams {
    const __nv_bfloat16 *bias;
    void *out;
    const uint32_t *mask;
    int mask_words;
    int expert_size;
    int32_t *status;
};

__device__ __forceinline__ float act_runtime(float z, int act)
{
    switch (act) {
    case D2D_ACT_RELU: return d2d_activate<D2D_ACT_RELU>(z);
    case D2D_ACT_GELU_ERF: return d2d_activate<D2D_ACT_GELU_ERF>(z);
    case D2D_ACT_GELU_TANH: return d2d_activate<D2D_ACT_GELU_TANH>(z);
    default: return d2d_activate<D2D_ACT_SILU>(z);
    }
}

// One CTA computes one 128 x BN tile.  GATED: two B tiles (gate, up) share the A tile and the
// epilogue combines A(gate) * (up + bias).
template <int BN, int STAGES, int EPI, bool GATED>
__global__ void __launch_bounds__(NTHREADS)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
               const __grid_constant__ CUtensorMap tm_b2, EpiParams ep, int M, int N, int K, int act)
{
    constexpr int A_BYTES = BM * BK * 2;
    constexpr int B_BYTES = BN * BK * 2;
    constexpr int STAGE_BYTES = A_BYTES + (GATED ? 2 : 1) * B_BYTES;
    constexpr int TMEM_COLS = GATED ? 2 * BN : BN;
    static_assert(TMEM_COLS == 32 || TMEM_COLS == 64 || TMEM_COLS == 128 || TMEM_COLS == 256 || TMEM_COLS == 512, "power of two");
    static_assert(BN % 32 == 0 && BN <= 256, "tile width");

    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);   // swizzle atoms are 1024-byte aligned
    __shared__ uint64_t bar_full[STAGES], bar_empty[STAGES], bar_acc;
    __shared__ uint32_t tmem_base_holder;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    const int nkb = (K + BK - 1) / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        mbar_init(smem_u32(&bar_acc), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_holder)),
                     "r"((uint32_t)TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_holder;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            for (int kb = 0; kb < nkb; ++kb) {
                const int s = kb % STAGES;
                const uint32_t round = (uint32_t)(kb / STAGES);
                if (!mbar_wait(smem_u32(&bar_empty[s]), (round & 1u) ^ 1u, ep.status)) break;
                const uint32_t full = smem_u32(&bar_full[s]);
                const uint32_t dst = smem_u32(smem + (size_t)s * STAGE_BYTES);
                mbar_expect_tx(full, (uint32_t)STAGE_BYTES);
                tma_load_2d(dst, &tm_a, kb * BK, m0, full);
                tma_load_2d(dst + A_BYTES, &tm_b, kb * BK, n0, full);
                if (GATED) tma_load_2d(dst + A_BYTES + B_BYTES, &tm_b2, kb * BK, n0, full);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = instr_desc_bf16(BM, BN);
            bool ok = true;
            for (int kb = 0; kb < nkb && ok; ++kb) {
                const int s = kb % STAGES;
                const uint32_t round = (uint32_t)(kb / STAGES);
                ok = mbar_wait(smem_u32(&bar_full[s]), round & 1u, ep.status);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t a_addr = smem_u32(smem + (size_t)s * STAGE_BYTES);
                const uint64_t da = smem_desc_sw128(a_addr);
                const uint64_t db = smem_desc_sw128(a_addr + A_BYTES);
                const uint64_t db2 = smem_desc_sw128(a_addr + A_BYTES + B_BYTES);
#pragma unroll
                for (int k = 0; k < BK / UMMA_K; ++k) {
                    const uint64_t koff = (uint64_t)((k * UMMA_K * 2) >> 4);    // 32 bytes per K step inside the swizzle row
                    const uint32_t accum = (kb | k) != 0 ? 1u : 0u;
                    umma_bf16(tmem_base, da + koff, db + koff, idesc, accum);
                    if (GATED) umma_bf16(tmem_base + BN, da + koff, db2 + koff, idesc, accum);
                }
                umma_commit(smem_u32(&bar_empty[s]));      // stage reusable once these MMAs have read it
            }
            umma_commit(smem_u32(&bar_acc));               // accumulator complete
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        const int quad = warp & 3;                          // TMEM lanes this warp may touch
        const int row = m0 + quad * 32 + lane;
        const bool acc_ok = mbar_wait(smem_u32(&bar_acc), 0, ep.status);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (acc_ok) {
            const uint32_t *mrow = (EPI == D2D_EPI_UP_MASKED && ep.mask && row < M)
                                       ? ep.mask + (size_t)row * ep.mask_words : nullptr;
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 32) {
                if (n0 + c0 >= N) break;                    // warp-uniform
                uint32_t r[32], g[32];
                const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)c0;
                tmem_ld32(taddr, r);
                if (GATED) tmem_ld32(taddr + BN, g);
                float v[32];
                int e = 0, rem = 0;
                if (EPI == D2D_EPI_UP_MASKED) {
                    e = (n0 + c0) / ep.expert_size;
                    rem = (n0 + c0) - e * ep.expert_size;
                }
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const int col = n0 + c0 + j;
                    const float b = (ep.bias && col < N) ? __bfloat162float(ep.bias[col]) : 0.0f;
                    float z = __uint_as_float(r[j]) + b;
                    if (EPI == D2D_EPI_RELU_BF16) z = fmaxf(z, 0.0f);
                    if (EPI == D2D_EPI_ABS_F32) z = fabsf(z);
                    if (EPI == D2D_EPI_UP_MASKED) {
                        bool keep = true;
                        if (mrow) keep = (mrow[e >> 5] >> (e & 31)) & 1u;
                        if (GATED) {
                            // first accumulator = up projection (+ bias), second = gate
                            z = keep ? act_runtime(__uint_as_float(g[j]), act) * z : 0.0f;
                        } else {
                            z = keep ? act_runtime(z, act) : 0.0f;
                        }
                        if (++rem == ep.expert_size) { rem = 0; ++e; }
                    }
                    v[j] = z;
                }
                if (row < M) {
                    const int col0 = n0 + c0;
                    if (EPI == D2D_EPI_ABS_F32) {
                        float *o = (float *)ep.out + (size_t)row * N + col0;
                        if (col0 + 32 <= N && (N & 3) == 0) {
#pragma unroll
                            for (int j = 0; j < 32; j += 4) *reinterpret_cast<float4 *>(o + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (col0 + j < N) o[j] = v[j];
                        }
                    } else {
                        __nv_bfloat16 *o = (__nv_bfloat16 *)ep.out + (size_t)row * N + col0;
                        if (col0 + 32 <= N && (N & 7) == 0) {
#pragma unroll
                            for (int j = 0; j < 32; j += 8) {
                                uint4 pk;
                                __nv_bfloat162 t0 = __floats2bfloat162_rn(v[j], v[j + 1]);
                                __nv_bfloat162 t1 = __floats2bfloat162_rn(v[j + 2], v[j + 3]);
                                __nv_bfloat162 t2 = __floats2bfloat162_rn(v[j + 4], v[j + 5]);
                                __nv_bfloat162 t3 = __floats2bfloat162_rn(v[j + 6], v[j + 7]);
                                pk.x = *reinterpret_cast<uint32_t *>(&t0);
                                pk.y = *reinterpret_cast<uint32_t *>(&t1);
                                pk.z = *reinterpret_cast<uint32_t *>(&t2);
                                pk.w = *reinterpret_cast<uint32_t *>(&t3);
                                *reinterpret_cast<uint4 *>(o + j) = pk;
                            }
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (col0 + j < N) o[j] = __float2bfloat16_rn(v[j]);
                        }
                    }
                }
            }
        }
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS) : "memory");
    }
}

// ------------------------------------------------------------------------------------------ host side

typedef CUresult (*encode_tiled_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                    const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

encode_tiled_fn get_encode()
{
    static encode_tiled_fn fn = [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return (encode_tiled_fn)p;
    }();
    return fn;
}

// [rows, cols] bf16 row-major matrix, box = box_rows x 64 columns, 128-byte swizzle, zero fill outside.
bool make_map(CUtensorMap *map, const void *base, int rows, int cols, int box_rows)
{
    encode_tiled_fn enc = get_encode();
    if (!enc) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BN, int STAGES, int EPI, bool GATED>
d2d_status launch(const d2d_gemm_args &g, cudaStream_t st)
{
    CUtensorMap ta, tb, tb2;
    if (!make_map(&ta, g.a, g.M, g.K, BM) || !make_map(&tb, g.b, g.N, g.K, BN)) return D2D_ERR_CUDA;
    if (GATED) {
        if (!make_map(&tb2, g.b_gate, g.N, g.K, BN)) return D2D_ERR_CUDA;
    } else {
        tb2 = tb;
    }
    constexpr int STAGE_BYTES = BM * BK * 2 + (GATED ? 2 : 1) * BN * BK * 2;
    constexpr size_t SMEM = (size_t)STAGES * STAGE_BYTES + 1024;
    auto kern = gemm_tc_kernel<BN, STAGES, EPI, GATED>;
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM) != cudaSuccess) return D2D_ERR_CUDA;
        attr_set = true;
    }
    EpiParams ep{(const __nv_bfloat16 *)g.bias, g.out, g.mask, g.mask_words, g.expert_size > 0 ? g.expert_size : 1, g.status};
    dim3 grid(d2d_cdiv(g.N, BN), d2d_cdiv(g.M, BM));
    kern<<<grid, NTHREADS, SMEM, st>>>(ta, tb, tb2, ep, g.M, g.N, g.K, g.act);
    D2D_LAUNCHED(1);
    return cudaGetLastError() == cudaSuccess ? D2D_OK : D2D_ERR_CUDA;
}

}  // namespace

bool d2d_gemm_tc_available() { return get_encode() != nullptr; }

d2d_status d2d_gemm_tc(const d2d_gemm_args &g, cudaStream_t st)
{
    if (g.M <= 0 || g.N <= 0 || g.K <= 0) return D2D_OK;
    if (g.K % 8) return D2D_ERR_UNSUPPORTED;
    switch (g.epilogue) {
    // 3 stages of 32 KB let two CTAs share an SM (one runs its epilogue while the other feeds the tensor cores)
    case D2D_EPI_RELU_BF16: return launch<128, 3, D2D_EPI_RELU_BF16, false>(g, st);
    case D2D_EPI_ABS_F32: return launch<128, 3, D2D_EPI_ABS_F32, false>(g, st);
    case D2D_EPI_BIAS_BF16: return launch<128, 3, D2D_EPI_BIAS_BF16, false>(g, st);
    case D2D_EPI_UP_MASKED:
        if (g.b_gate) return launch<128, 4, D2D_EPI_UP_MASKED, true>(g, st);
        return launch<128, 3, D2D_EPI_UP_MASKED, false>(g, st);
    }
    return D2D_ERR_INVALID_ARG;
}
