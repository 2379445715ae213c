// Inline-PTX building blocks shared by the tensor-core kernels (tcgen05.mma with TMEM accumulators, TMA tile
// loads, mbarrier pipelines) and the activation math of their epilogues.  Everything here is a per-CTA operation;
// no load is shared between CTAs.
#pragma once

#include <cuda.h>

#include "d2d_common.cuh"

namespace d2d_tc {

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
// Bounded wait for the phase with the given parity; false (and status set) when the limit runs out.  SPIN polls run
// back to back, later ones are SLEEP nanoseconds apart.
template <int SPIN = 64, int SLEEP = 32>
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
        if (it > (uint32_t)SPIN) __nanosleep(SLEEP);
    }
    if (status) atomicMax(status, (int32_t)D2D_ERR_TIMEOUT);
    return false;
}

// One non-blocking test of the phase with the given parity.
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity)
{
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    return done != 0;
}

// Bounded wait for whole warps: try_wait may suspend the warp in hardware until the phase completes or a time
// limit passes, so thirty-two waiting lanes cost no issue slots.  Nothing in the loop depends on the lane (same
// barrier, same parity, the timer is read by one warp instruction), so the lanes stay in step and take the same
// decision; a vote at the end would make that explicit but measured 1.8 % slower on the ViT-shaped layer.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, int32_t *status)
{
    // how long one try may suspend is up to the hardware, so the bound is in time: about a second by the global timer
    unsigned long long t0 = 0;
    for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(bar), "r"(parity)
            : "memory");
        if (done) return true;
        if ((it & 31u) == 31u) {                               // rarely reached: a try normally ends with the phase complete
            unsigned long long now;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
            if (t0 == 0) t0 = now;
            else if (now - t0 > 1000000000ull) break;
        }
    }
    if (status) atomicMax(status, (int32_t)D2D_ERR_TIMEOUT);
    return false;
}
// true in exactly one lane of a converged warp
__device__ __forceinline__ bool elect_one()
{
    uint32_t pred;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "elect.sync _|p, 0xffffffff;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(pred));
    return pred != 0;
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
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Activations of the bf16 tensor-core path.  Results are rounded to bf16 (8 bits of mantissa,
// 2^-9 relative), and the epilogue of the up projection is issue-bound (K = d is short compared
// with the 128 x BN outputs of a tile), so every activation is built on ONE special-function
// instruction, the hardware tanh (relative error about 2^-11):
//   SiLU       z * sigmoid(z)            = z * (0.5 + 0.5 tanh(z / 2))
//   GELU tanh  0.5 z (1 + tanh(c (z + 0.044715 z^3)))
//   GELU erf   0.5 z (1 + erf(z / sqrt 2)),  erf(z / sqrt 2) ~= tanh(z (a + b z^2 + c z^4)), a quintic
//              argument fitted to erf with maximum error 3.7e-5 (GELU: 5.4e-5 absolute before the tanh
//              instruction's own error) -- well below what a bf16 result can represent.
__device__ __forceinline__ float fast_tanh(float x)
{
    float y;
    asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int ACT> __device__ __forceinline__ float fast_act(float z)
{
    if (ACT == D2D_ACT_RELU) return fmaxf(z, 0.0f);
    if (ACT == D2D_ACT_GELU_ERF) {
        // the quintic was fitted on |z| <= 8 and turns over beyond |z| ~ 11: clamp z^2 inside it (tanh is 1 there anyway)
        const float z2 = fminf(z * z, 64.0f);
        const float q = fmaf(fmaf(-3.15807042e-4f, z2, 3.67982560e-2f), z2, 7.97717834e-1f);
        const float t = fast_tanh(z * q);
        return z * fmaf(0.5f, t, 0.5f);
    }
    if (ACT == D2D_ACT_GELU_TANH) {
        const float q = fmaf(0.79788456080286536f * 0.044715f, z * z, 0.79788456080286536f);
        const float t = fast_tanh(z * q);
        return z * fmaf(0.5f, t, 0.5f);
    }
    const float t = fast_tanh(0.5f * z);                   // SiLU
    return z * fmaf(0.5f, t, 0.5f);
}

// ---- packed float32 pairs (sm_100 issues add / mul / fma on two float32 values per instruction; same IEEE results
// as the scalar forms).  The epilogue is bound by instruction issue, so its per-element math runs on pairs.
__device__ __forceinline__ uint64_t pack2(float a, float b)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float &a, float &b) { asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v)); }
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b)
{
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b)
{
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t dup2(float a) { return pack2(a, a); }

// fast_act on a pair; the same operations in the same order as the scalar form, so the results are identical
template <int ACT> __device__ __forceinline__ uint64_t fast_act2(uint64_t z)
{
    float a, b;
    if (ACT == D2D_ACT_RELU) {
        unpack2(z, a, b);
        return pack2(fmaxf(a, 0.0f), fmaxf(b, 0.0f));
    }
    uint64_t arg;
    if (ACT == D2D_ACT_GELU_ERF) {
        unpack2(mul2(z, z), a, b);
        const uint64_t z2 = pack2(fminf(a, 64.0f), fminf(b, 64.0f));
        const uint64_t q = fma2(fma2(dup2(-3.15807042e-4f), z2, dup2(3.67982560e-2f)), z2, dup2(7.97717834e-1f));
        arg = mul2(z, q);
    } else if (ACT == D2D_ACT_GELU_TANH) {
        const uint64_t q = fma2(dup2(0.79788456080286536f * 0.044715f), mul2(z, z), dup2(0.79788456080286536f));
        arg = mul2(z, q);
    } else {
        arg = mul2(dup2(0.5f), z);                          // SiLU
    }
    unpack2(arg, a, b);
    const uint64_t t = pack2(fast_tanh(a), fast_tanh(b));
    return mul2(z, fma2(dup2(0.5f), t, dup2(0.5f)));
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
}

}  // namespace d2d_tc

// ---- host side (defined in gemm_tc.cu) ----
// [rows, cols] bf16 row-major matrix as a TMA tensor map: box = box_rows x 64 columns, 128-byte swizzle, zero fill
// outside the matrix.  False when the driver entry point for tensor-map encoding is unavailable or the encode fails.
bool d2d_tc_make_map(CUtensorMap *map, const void *base, int rows, int cols, int box_rows);
// Number of SMs of the current device (148 when the query fails).
int d2d_tc_sm_count();
// False when D2D_GEMM_PDL=0 asks for fully serialised launches.
bool d2d_tc_pdl_enabled();
