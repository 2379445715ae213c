// bf16 GEMM C[M,N] = epilogue(A[M,K] B[N,K]^T) on the 5th-generation tensor cores of sm_100a.
//
//   warp 0   TMA producer: cp.async.bulk.tensor tiles of A (128 x 64) and B (BN x 64), 128-byte
//            swizzled, into a ring of shared-memory stages guarded by full/empty mbarriers
//   warp 1   allocates TMEM and issues tcgen05.mma (one thread), fp32 accumulators in TMEM
//            (two buffers); tcgen05.commit releases a stage when the MMAs that read it have retired
//   warps 2-17 epilogue: tcgen05.ld the accumulator (one row per thread), bias / activation /
//            selection mask, vectorised stores; runs while the next tile's MMAs fill the other buffer
// The kernel is persistent: one CTA per SM walks over the output tiles.
//
// Every mbarrier wait is bounded: when the limit runs out the role records D2D_ERR_TIMEOUT in the
// status word and leaves its loop, all roles meet at the final barrier, TMEM is freed and the
// kernel returns (no trap, no endless spin).  Every load is a plain per-CTA load.
#include "gemm_tc.cuh"
#include "tc_common.cuh"

#include <stdlib.h>

namespace {

using namespace d2d_tc;

constexpr int BM = 128;          // rows of A per CTA = TMEM lanes
constexpr int BK = 64;           // 64 bf16 = one 128-byte swizzle row
constexpr int UMMA_K = 16;

struct EpiParams {
    const __nv_bfloat16 *bias;
    void *out;
    const uint32_t *mask;
    int mask_words;
    int expert_size;
    int32_t *status;
    uint32_t inv_expert_size;        // ceil(2^32 / expert_size): column / expert_size = umulhi(column, inv) for columns < 2^16
    int *tile_counter;               // device counter (zero at launch) for dynamic tile scheduling, NULL = static round-robin
    int late_wait;                   // 1: only the epilogue waits for the previous kernel of the stream (see below)
    int gate_cat;                    // 1 (gated): tm_b covers up and gate rows interleaved in blocks of BN, one load brings both
    int band_rows;                   // > 0: tiles are walked column-major inside bands of this many row tiles (L2 reuse)
    int batch;                       // >= 1 problems of one shape: A columns, B rows, bias entries and out advance per problem
    const int32_t *n_sel;            // density-adaptive dispatch: do nothing when *n_sel <= n_sel_max (NULL: always run)
    long long n_sel_max;
    int test_skip_load;              // test aid: CTA 0 never requests the A tile of its first k-block (see d2d_gemm_args)
};

// Tile index -> (row tile, column tile).  Plain order is row-major: CTAs that run together share a few rows of A and
// sweep all of B, so B is streamed from HBM once per wave when A and B together exceed L2.  With bands, the tiles of
// `band` consecutive row tiles are walked column by column: the band's rows of A stay in L2 while B is streamed once
// per band.
__device__ __forceinline__ void tile_coords(int tile, int rows, int cols, int band, int &r, int &c)
{
    if (band <= 0) { r = tile / cols; c = tile - r * cols; return; }
    const int per_band = band * cols;
    const int b = tile / per_band, idx = tile - b * per_band;
    const int h = rows - b * band < band ? rows - b * band : band;      // height of this band (the last may be short)
    c = idx / h;
    r = b * band + (idx - c * h);
}


// 16 accumulator columns -> 16 output values: bias (float32, staged in shared memory), activation, selection mask.
template <int EPI, int ACT, bool GATED>
__device__ __forceinline__ void epilogue_16(const uint32_t (&r)[16], const uint32_t (&g)[16], float (&v)[16],
                                            const float *bias_f, bool has_bias, int col0, uint32_t keep, bool halves)
{
    float bias[16];
    if (has_bias) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const float4 b4 = *reinterpret_cast<const float4 *>(bias_f + col0 + 4 * q);
            bias[4 * q] = b4.x; bias[4 * q + 1] = b4.y; bias[4 * q + 2] = b4.z; bias[4 * q + 3] = b4.w;
        }
    } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) bias[j] = 0.0f;
    }
    if (EPI == D2D_EPI_UP_MASKED && halves) {
        // the common case of the up projection: math on pairs; the selection is applied by the caller on the packed
        // bf16 words (each 8-column half belongs to one expert)
#pragma unroll
        for (int j = 0; j < 16; j += 2) {
            // first accumulator = up projection (+ bias), second = gate
            const uint64_t z = add2(pack2(__uint_as_float(r[j]), __uint_as_float(r[j + 1])), pack2(bias[j], bias[j + 1]));
            const uint64_t h = GATED ? mul2(fast_act2<ACT>(pack2(__uint_as_float(g[j]), __uint_as_float(g[j + 1]))), z)
                                     : fast_act2<ACT>(z);
            unpack2(h, v[j], v[j + 1]);
        }
        return;
    }
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        float z = __uint_as_float(r[j]) + bias[j];
        if (EPI == D2D_EPI_RELU_BF16) z = fmaxf(z, 0.0f);
        if (EPI == D2D_EPI_ABS_F32) z = fabsf(z);
        if (EPI == D2D_EPI_UP_MASKED) {
            const float h = GATED ? fast_act<ACT>(__uint_as_float(g[j])) * z : fast_act<ACT>(z);
            z = ((keep >> j) & 1u) ? h : 0.0f;
        }
        v[j] = z;
    }
}

// Same result with every bound checked (ragged last column tile, odd leading dimension, bias too long for the cache).
// Statically indexed and inlined: an out-of-line version forced the accumulator registers onto the stack.
template <int EPI, int ACT, bool GATED>
__device__ __forceinline__ void epilogue_16_slow(const uint32_t (&r)[16], const uint32_t (&g)[16], const __nv_bfloat16 *bias,
                                                 void *out, int row, int M, int col0, int N, uint32_t keep)
{
    if (row >= M) return;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        if (col0 + j < N) {
            float z = __uint_as_float(r[j]) + (bias ? __bfloat162float(bias[col0 + j]) : 0.0f);
            if (EPI == D2D_EPI_RELU_BF16) z = fmaxf(z, 0.0f);
            if (EPI == D2D_EPI_ABS_F32) z = fabsf(z);
            if (EPI == D2D_EPI_UP_MASKED) {
                const float h = GATED ? fast_act<ACT>(__uint_as_float(g[j])) * z : fast_act<ACT>(z);
                z = ((keep >> j) & 1u) ? h : 0.0f;
            }
            if (EPI == D2D_EPI_PARTIAL_F32) atomicAdd((float *)out + (size_t)row * N + col0 + j, z);
            else if (EPI == D2D_EPI_ABS_F32) ((float *)out)[(size_t)row * N + col0 + j] = z;
            else ((__nv_bfloat16 *)out)[(size_t)row * N + col0 + j] = __float2bfloat16_rn(z);
        }
    }
}

constexpr int N_EPI_WARPS = 16;
constexpr int BIAS_CACHE_ELEMS = 6144;           // 24 KB of float32 in shared memory behind the operand stages
constexpr int NTHREADS_V2 = 64 + 32 * N_EPI_WARPS;

__host__ __device__ constexpr int pow2_at_least(int v) { return v <= 32 ? 32 : v <= 64 ? 64 : v <= 128 ? 128 : v <= 256 ? 256 : 512; }

// Persistent kernel: CTA c computes tiles c, c + gridDim.x, ... (128 x BN each, column tiles
// fastest).  Two accumulator buffers in TMEM let the epilogue of one tile overlap the MMAs of the
// next.  GATED: two B tiles (up, gate) share the A tile; the epilogue forms A(gate) * (up + bias).
template <int BN, int STAGES, int EPI, int ACT, bool GATED>
__global__ void __launch_bounds__(NTHREADS_V2, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
               const __grid_constant__ CUtensorMap tm_b2, EpiParams ep, int M, int N, int K, int k_splits)
{
    constexpr int TM = BM;                                // rows of the tile a CTA computes
    constexpr int B_ROWS = BN;                            // rows of B this CTA stages
    constexpr int A_BYTES = BM * BK * 2;
    constexpr int B_BYTES = B_ROWS * BK * 2;
    constexpr int STAGE_BYTES = A_BYTES + (GATED ? 2 : 1) * B_BYTES;
    constexpr int BUF_COLS = pow2_at_least(GATED ? 2 * BN : BN);    // TMEM columns per accumulator buffer
    constexpr int TMEM_COLS = 2 * BUF_COLS;
    constexpr int COLS_PER_WARP = BN / 4;                            // four epilogue warps share a TMEM lane quadrant
    static_assert(TMEM_COLS <= 512 && BN % 64 == 0 && BN <= 256, "tile width");

    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);   // swizzle atoms are 1024-byte aligned
    __shared__ uint64_t bar_full[STAGES], bar_empty[STAGES], bar_acc_full[2], bar_acc_empty[2];
    __shared__ uint32_t tmem_base_holder;
    __shared__ volatile int epi_ok[2];                               // outcome of the epilogue's accumulator wait (per buffer parity)
    // dynamic scheduling: the producer draws work items from a global counter and hands them to the MMA thread and
    // to the epilogue through a two-slot ring (a CTA that starts late, or gets slow tiles, simply draws fewer)
    __shared__ uint64_t sched_full[2], sched_empty[2];
    __shared__ volatile int sched_item[2], epi_item[2];
    constexpr int MASK_REGS = 8;                                     // selection words of a row kept in registers (E <= 256; wider masks are read through L1)
    // the whole bias vector is staged once, as float32, behind the operand stages when it fits
    float *bias_f = reinterpret_cast<float *>(smem + (size_t)STAGES * STAGE_BYTES);
    const int NB = N * ep.batch;                                     // bias entries of all problems
    const bool bias_cached = ep.bias != nullptr && NB <= BIAS_CACHE_ELEMS && (N & 3) == 0;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nkb = (K + BK - 1) / BK;
    const int n_tiles = (N + BN - 1) / BN;
    // work item = (output tile, K split); with k_splits > 1 every item accumulates a slice of K and the
    // epilogue adds its partial sums to a float32 buffer (small-M problems that would leave most SMs idle)
    const int tiles_pp = ((M + TM - 1) / TM) * n_tiles;            // output tiles per problem
    const int total_tiles = tiles_pp * ep.batch * k_splits;
    const int worker = (int)blockIdx.x;
    const int n_workers = (int)gridDim.x;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&bar_acc_full[b]), 1);
            mbar_init(smem_u32(&bar_acc_empty[b]), N_EPI_WARPS);
            mbar_init(smem_u32(&sched_full[b]), 1);
            mbar_init(smem_u32(&sched_empty[b]), 2);          // read by the MMA thread and by the epilogue's leader
        }
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
    // Programmatic dependent launch: everything above (barriers, TMEM, the bias vector: parameters, not activations)
    // may run while the previous kernel of the stream drains; nothing below starts before that kernel has completed
    // and its writes are visible.  The next kernel of the stream may be scheduled onto SMs as this grid frees them.
    // With late_wait only the epilogue depends on that kernel (the selection mask written by the router): the
    // operand loads and the MMAs of the first tiles then overlap it, and only the epilogue warps wait.
    const bool dyn = ep.tile_counter != nullptr;
    if (bias_cached && warp >= 2) {
        // The epilogue warps stage the bias (a parameter: no need to wait for the previous kernel) while the producer
        // and the MMA thread are already at work.  16-byte loads, all issued before the first use: the fill costs one
        // memory latency, not N / threads of them.
        for (int i = ((int)threadIdx.x - 64) * 8; i < NB; i += N_EPI_WARPS * 32 * 8) {
            float b8[8];
            if (i + 8 <= NB) {
                d2d_load8(ep.bias + i, b8);
#pragma unroll
                for (int q = 0; q < 8; ++q) bias_f[i + q] = b8[q];
            } else {
                for (int q = 0; i + q < NB; ++q) bias_f[i + q] = __bfloat162float(ep.bias[i + q]);
            }
        }
        asm volatile("bar.sync 1, %0;" ::"r"(N_EPI_WARPS * 32) : "memory");
    }
    // early_b: the B operand (weights) does not depend on the previous kernel either, so the producer requests the B
    // tiles of its first k-blocks BEFORE it waits for that kernel and only the A tiles after (static schedule only)
    const bool early_b = !dyn && !ep.late_wait && ep.n_sel == nullptr;
    if (warp >= 2 || (!ep.late_wait && !(early_b && warp == 0))) asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // density-adaptive dispatch: below the crossover the gathered kernel, launched next to this one, does the work
    // (every thread has passed the dependency wait here: the host never combines n_sel with late_wait)
    const bool run = ep.n_sel == nullptr || (long long)__ldcg(ep.n_sel) > ep.n_sel_max;

    if (!run) {
        // nothing to do
    } else if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t it = 0, pre = 0;
            bool ok = true;
            // B tile(s) of k-block kb into the stage at dst (single-CTA form)
            auto load_b = [&](uint32_t dst, uint32_t full, int kb, int n0) {
                if (GATED && ep.gate_cat) {
                    // up rows [n0, n0+BN) and gate rows [n0, n0+BN) are adjacent in the interleaved copy: one
                    // 2*BN-row box (the producer thread's time per k-block is what bounds the gated main loop)
                    tma_load_2d(dst + A_BYTES, &tm_b, kb * BK, 2 * n0, full);
                } else {
                    tma_load_2d(dst + A_BYTES, &tm_b, kb * BK, n0, full);
                    if (GATED) tma_load_2d(dst + A_BYTES + B_BYTES, &tm_b2, kb * BK, n0, full);
                }
            };
            for (uint32_t local = 0; ok; ++local) {
                int item = worker + (int)local * n_workers;
                if (dyn) {
                    const uint32_t sl = local & 1u, use = local >> 1;
                    ok = mbar_wait(smem_u32(&sched_empty[sl]), (use & 1u) ^ 1u, ep.status);
                    if (!ok) break;
                    // A CTA's first item is its own index (no round trip to the counter before the first loads); the
                    // counter hands out the items from gridDim.x on.  Every CTA draws exactly one value past the end,
                    // total_tiles draws in all: whoever gets the last one leaves the counter at zero for the next launch.
                    if (local > 0) {
                        const int c = atomicAdd(ep.tile_counter, 1);
                        if (c == total_tiles - 1) *ep.tile_counter = 0;
                        item = (int)gridDim.x + c;
                    }
                    sched_item[sl] = item < total_tiles ? item : -1;
                    mbar_arrive(smem_u32(&sched_full[sl]));       // release: the slot's content is visible to whoever sees the phase
                }
                if (item >= total_tiles) break;
                int tile = (!GATED && k_splits == 1) ? item : item / k_splits;
                const int sp = item - tile * k_splits;
                // no split is the common case: skip the divisions (measured: faster for the plain kernels, slower for the
                // gated one, whose code layout is at its limit)
                const bool one = !GATED && k_splits == 1;
                const int kb0 = one ? 0 : (int)((long long)sp * nkb / k_splits), kb1 = one ? nkb : (int)((long long)(sp + 1) * nkb / k_splits);
                int prob = 0;
                if (ep.batch > 1) { prob = tile / tiles_pp; tile -= prob * tiles_pp; }
                int tr, tc;
                tile_coords(tile, (M + TM - 1) / TM, n_tiles, ep.band_rows, tr, tc);
                const int m0 = tr * TM, n0 = prob * N + tc * BN;
                const int ka = prob * K;                      // problem p reads columns [p*K, (p+1)*K) of A
                if (early_b && local == 0) {
                    // arm the first stages and request their B tiles, then wait for the previous kernel (A may be its output)
                    for (int kb = kb0; kb < kb1 && pre < (uint32_t)STAGES; ++kb, ++pre) {
                        const uint32_t full = smem_u32(&bar_full[pre]);
                        mbar_expect_tx(full, (uint32_t)STAGE_BYTES);
                        load_b(smem_u32(smem + (size_t)pre * STAGE_BYTES), full, kb, n0);
                    }
                    asm volatile("griddepcontrol.wait;" ::: "memory");
                }
                for (int kb = kb0; kb < kb1; ++kb, ++it) {
                    const uint32_t s = it % STAGES, round = it / STAGES;
                    if (it < pre) {                           // armed above, B already requested
                        // host-made fault for the failure-handling test: this stage's byte count is never reached, so the
                        // MMA warp's wait, then the epilogue's and this thread's own, run out and the CTA leaves in order
                        if (ep.test_skip_load && it == 0 && blockIdx.x == 0) continue;
                        tma_load_2d(smem_u32(smem + (size_t)s * STAGE_BYTES), &tm_a, ka + kb * BK, m0, smem_u32(&bar_full[s]));
                        continue;
                    }
                    ok = mbar_wait(smem_u32(&bar_empty[s]), (round & 1u) ^ 1u, ep.status);
                    if (!ok) break;
                    const uint32_t dst = smem_u32(smem + (size_t)s * STAGE_BYTES);
                    const uint32_t full = smem_u32(&bar_full[s]);
                    mbar_expect_tx(full, (uint32_t)STAGE_BYTES);
                    tma_load_2d(dst, &tm_a, ka + kb * BK, m0, full);
                    load_b(dst, full, kb, n0);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        // The whole warp walks the loop, so that waits, indices and descriptors are warp-uniform (the tensor-core
        // instructions take their operands from uniform registers); one elected lane issues the MMAs and commits.
        {
            // Gated: the up and gate tiles sit back to back in shared memory, so they are ONE K-major
            // B operand of 2*BN rows and one MMA fills both accumulators (columns [0,BN) up, [BN,2BN) gate).
            // Two N=BN instructions would each pay the full A-operand read and run at half the rate.
            const uint32_t idesc = instr_desc_bf16(TM, GATED ? 2 * BN : BN);
            uint32_t it = 0, local = 0;
            bool ok = true;
            // The tensor core accepts only a few instructions ahead, so whatever this thread executes between the last
            // MMA of one k-block and the first MMA of the next is a bubble in the MMA pipe.  The barrier of the NEXT
            // k-block is therefore tested between the MMAs of the current one (`have` carries the answer across
            // k-blocks and tiles), and nothing but the commit sits between two k-blocks whose data has landed.
            bool have = false;
            for (;; ++local) {
                int item = worker + (int)local * n_workers;
                if (dyn) {
                    const uint32_t sl = local & 1u, su = local >> 1;
                    ok = mbar_wait_warp(smem_u32(&sched_full[sl]), su & 1u, ep.status);
                    if (!ok) break;
                    item = sched_item[sl];
                    __syncwarp();                              // every lane has read the slot before it is handed back
                    if (elect_one()) mbar_arrive(smem_u32(&sched_empty[sl]));
                    if (item < 0) break;
                }
                if (item >= total_tiles) break;
                const int sp = (!GATED && k_splits == 1) ? 0 : item % k_splits;
                // no split is the common case: skip the divisions (measured: faster for the plain kernels, slower for the
                // gated one, whose code layout is at its limit)
                const bool one = !GATED && k_splits == 1;
                const int kb0 = one ? 0 : (int)((long long)sp * nkb / k_splits), kb1 = one ? nkb : (int)((long long)(sp + 1) * nkb / k_splits);
                const uint32_t buf = local & 1u, use = local >> 1;
                ok = mbar_wait_warp(smem_u32(&bar_acc_empty[buf]), (use & 1u) ^ 1u, ep.status);   // epilogue drained this buffer
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t acc = tmem_base + buf * BUF_COLS;
                for (int kb = kb0; kb < kb1; ++kb, ++it) {
                    const uint32_t s = it % STAGES, round = it / STAGES;
                    if (!have) {
                        ok = mbar_wait_warp(smem_u32(&bar_full[s]), round & 1u, ep.status);
                        if (!ok) break;
                    }
                    const uint32_t a_addr = smem_u32(smem + (size_t)s * STAGE_BYTES);
                    const uint64_t da = smem_desc_sw128(a_addr);
                    const uint64_t db = smem_desc_sw128(a_addr + A_BYTES);
                    const uint64_t db2 = smem_desc_sw128(a_addr + A_BYTES + B_BYTES);
                    const uint32_t s_next = (it + 1) % STAGES, round_next = (it + 1) / STAGES;
                    auto issue = [&](int k) {
                        const uint64_t koff = (uint64_t)((k * UMMA_K * 2) >> 4);    // 32 bytes per K step inside the swizzle row
                        const uint32_t accum = (kb > kb0 || k != 0) ? 1u : 0u;
                        umma_bf16(acc, da + koff, db + koff, idesc, accum);
                    };
                    if (elect_one()) {
#pragma unroll
                        for (int k = 0; k < BK / UMMA_K - 1; ++k) issue(k);
                    }
                    // before the last MMA of this k-block: has the next k-block (of this or the next tile) landed?
                    have = __all_sync(0xffffffffu, mbar_test(smem_u32(&bar_full[s_next]), round_next & 1u));
                    if (elect_one()) {
                        issue(BK / UMMA_K - 1);
                        umma_commit(smem_u32(&bar_empty[s]));        // stage reusable once these MMAs have read it
                    }
                    __syncwarp();
                }
                if (!ok) break;
                if (elect_one()) umma_commit(smem_u32(&bar_acc_full[buf]));   // accumulator of this tile complete
                __syncwarp();
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..17)
        // Sixteen warps (four per TMEM lane quadrant) so that the per-element math of one warp hides
        // the TMEM-load and MUFU latencies of another.  A warp walks its BN/4 columns in 16-column
        // units; the load of the next unit is in flight while the current one is processed, and the
        // rarely taken paths are out of line so that the unrolled body stays small (a 32-column,
        // everything-inline version of this epilogue was instruction-fetch bound).
        const int ew = warp - 2;
        const int quad = warp & 3;                          // TMEM lanes this warp may touch
        const int part = ew >> 2;                           // which quarter of the tile's columns
        constexpr int N_UNITS = COLS_PER_WARP / 16;
        uint32_t local = 0;
        bool ok = true;
        for (;; ++local) {
            const uint32_t buf = local & 1u, use = local >> 1;
            int item = worker + (int)local * n_workers;
            if (dyn) {
                // the leader takes the item from the ring and publishes it to the sixteen warps
                if (ew == 0 && lane == 0) {
                    int got = -2;                            // -2: the wait ran out
                    if (mbar_wait(smem_u32(&sched_full[buf]), use & 1u, ep.status)) {
                        got = sched_item[buf];
                        mbar_arrive(smem_u32(&sched_empty[buf]));
                    }
                    epi_item[buf] = got;
                }
                asm volatile("bar.sync 1, %0;" ::"r"(N_EPI_WARPS * 32) : "memory");
                item = epi_item[buf];
                if (item < 0) break;
            }
            if (item >= total_tiles) break;
            int tile = (!GATED && k_splits == 1) ? item : item / k_splits;
            int prob = 0;
            if (ep.batch > 1) { prob = tile / tiles_pp; tile -= prob * tiles_pp; }
            int tr, tc;
            tile_coords(tile, (M + TM - 1) / TM, n_tiles, ep.band_rows, tr, tc);
            const int m0 = tr * TM, n0 = tc * BN;
            // this problem's bias entries and output matrix
            const float *bias_p = bias_f + prob * N;
            const __nv_bfloat16 *bias_g = ep.bias ? ep.bias + prob * N : nullptr;
            void *out_p = (char *)ep.out + (size_t)prob * M * N * ((EPI == D2D_EPI_ABS_F32 || EPI == D2D_EPI_PARTIAL_F32) ? 4 : 2);
            const int row = m0 + quad * 32 + lane;
            // this row's selection words go to registers before the wait, so their latency is hidden
            uint32_t mw[MASK_REGS];
            const uint32_t *mrow = nullptr;
            if (EPI == D2D_EPI_UP_MASKED && ep.mask && row < M) {
                mrow = ep.mask + (size_t)row * ep.mask_words;
                if (ep.mask_words <= MASK_REGS) {
#pragma unroll
                    for (int i = 0; i < MASK_REGS; ++i) mw[i] = i < ep.mask_words ? __ldg(mrow + i) : 0u;
                }
            }
            // ONE thread polls the accumulator barrier and the other epilogue warps sleep on a hardware barrier: sixteen
            // pollers measurably slow the producer and MMA threads, whose own barrier tests share the same unit
            if (ew == 0 && lane == 0) epi_ok[local & 1u] = mbar_wait(smem_u32(&bar_acc_full[buf]), use & 1u, ep.status) ? 1 : 0;
            asm volatile("bar.sync 1, %0;" ::"r"(N_EPI_WARPS * 32) : "memory");
            ok = epi_ok[local & 1u] != 0;
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t tbase = tmem_base + buf * BUF_COLS + ((uint32_t)(quad * 32) << 16) + (uint32_t)(part * COLS_PER_WARP);

            // expert that owns the first column of this warp's range (one division per tile; advanced incrementally)
            const int colw = n0 + part * COLS_PER_WARP;
            int e = 0, lo = 0, widx = -1;
            uint32_t word = 0u;
            if (EPI == D2D_EPI_UP_MASKED && mrow) {
                e = colw / ep.expert_size;
                lo = e * ep.expert_size - colw;             // first column of expert e relative to the current unit (<= 0)
            }
            const bool bias_fast = ep.bias == nullptr || bias_cached;
            const bool wide_store = (N & 15) == 0 && (reinterpret_cast<uintptr_t>(out_p) & 31) == 0;   // 32-byte aligned rows
            const bool mask_on = EPI == D2D_EPI_UP_MASKED && ep.mask != nullptr;                         // CTA-uniform
            // The common case gets a loop of its own with nothing else in it (the epilogue is sensitive to its
            // instruction-cache footprint): a full-width tile, the bias in shared memory, vector-aligned rows and
            // expert sizes that are multiples of 8.  Everything else (ragged last column tile, odd sizes, a bias too
            // long for the cache) goes through the compact generic loop below.
            const bool fast_tile = bias_fast && (N & 7) == 0 && n0 + BN <= N && (!mask_on || (ep.expert_size & 7) == 0);
            uint32_t ra[16], rb[GATED ? 1 : 16], ga[GATED ? 16 : 1];
            if (fast_tile) {
                // Non-gated: the next unit's accumulators are prefetched into a second register set.  Gated tiles need
                // two accumulators per column; a second set would spill, so each unit is loaded when it is needed and
                // the other epilogue warps of the SM sub-partition cover the latency.
                if (!GATED) tmem_ld16_issue(tbase, ra);
                // selection bits of this row, one per 8-column group of the warp's columns (each group belongs to one
                // expert; e = col / s by a multiply-high with the precomputed reciprocal); done once per tile so that the
                // unrolled units below stay small
                uint32_t kbits = 0xffffffffu;
                if (mask_on && mrow) {
                    kbits = 0u;
#pragma unroll
                    for (int h = 0; h < COLS_PER_WARP / 8; ++h) {
                        const uint32_t ee = __umulhi((uint32_t)(colw + 8 * h), ep.inv_expert_size);
                        const int wi = (int)(ee >> 5);
                        uint32_t wd;
                        if (ep.mask_words <= MASK_REGS) {
                            wd = mw[0];
#pragma unroll
                            for (int i = 1; i < MASK_REGS; ++i) wd = (i == wi) ? mw[i] : wd;
                        } else {
                            wd = __ldg(mrow + wi);
                        }
                        kbits |= ((wd >> (ee & 31)) & 1u) << h;
                    }
                }
#pragma unroll
                for (int u = 0; u < N_UNITS; ++u) {             // at most 4 units
                    const int col0 = colw + u * 16;
                    uint32_t (&r)[16] = GATED ? ra : ((u & 1) ? reinterpret_cast<uint32_t (&)[16]>(rb) : ra);
                    uint32_t (&g)[16] = reinterpret_cast<uint32_t (&)[16]>(ga);
                    if (GATED) {
                        tmem_ld16_issue(tbase + u * 16, ra);
                        tmem_ld16_issue(tbase + u * 16 + BN, reinterpret_cast<uint32_t (&)[16]>(ga));
                    }
                    const uint32_t keep = ((kbits >> (2 * u)) & 1u ? 0x00ffu : 0u) | ((kbits >> (2 * u + 1)) & 1u ? 0xff00u : 0u);
                    tmem_ld_wait();                                               // this unit's accumulators have landed
                    if (!GATED && u + 1 < N_UNITS)                                // the next unit's load overlaps the math below
                        tmem_ld16_issue(tbase + (u + 1) * 16, (u & 1) ? ra : reinterpret_cast<uint32_t (&)[16]>(rb));

                    float v[16];
                    epilogue_16<EPI, ACT, GATED>(r, g, v, bias_p, ep.bias != nullptr, col0, keep, EPI == D2D_EPI_UP_MASKED);
                    if (row < M) {
                        if (EPI == D2D_EPI_PARTIAL_F32) {
                            float *o = (float *)out_p + (size_t)row * N + col0;
#pragma unroll
                            for (int j = 0; j < 16; j += 4)
                                asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(o + j), "f"(v[j]), "f"(v[j + 1]),
                                             "f"(v[j + 2]), "f"(v[j + 3]) : "memory");
                        } else if (EPI == D2D_EPI_ABS_F32) {
                            float *o = (float *)out_p + (size_t)row * N + col0;
#pragma unroll
                            for (int j = 0; j < 16; j += 4) *reinterpret_cast<float4 *>(o + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                        } else {
                            __nv_bfloat16 *o = (__nv_bfloat16 *)out_p + (size_t)row * N + col0;
                            uint32_t pk[8];
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                __nv_bfloat162 t = __floats2bfloat162_rn(v[2 * j], v[2 * j + 1]);
                                pk[j] = *reinterpret_cast<uint32_t *>(&t);
                                // selection: an expert the token did not keep contributes zeros (also when its
                                // pre-activations are not finite)
                                if (EPI == D2D_EPI_UP_MASKED) pk[j] = (keep >> (2 * j)) & 1u ? pk[j] : 0u;
                            }
                            if (wide_store) {
                                // one 32-byte store per row and unit: a whole sector per lane, half as many store instructions
                                asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(o), "r"(pk[0]), "r"(pk[1]),
                                             "r"(pk[2]), "r"(pk[3]), "r"(pk[4]), "r"(pk[5]), "r"(pk[6]), "r"(pk[7]) : "memory");
                            } else {
                                *reinterpret_cast<uint4 *>(o) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                                *reinterpret_cast<uint4 *>(o + 8) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
                            }
                        }
                    }
                }
            } else {
                // generic loop: one unit at a time, every bound checked, any expert size
                uint32_t (&g)[16] = reinterpret_cast<uint32_t (&)[16]>(ga);
#pragma unroll 1
                for (int u = 0; u < N_UNITS; ++u) {
                    const int col0 = colw + u * 16;
                    if (col0 >= N) break;                       // warp-uniform (ragged last column tile)
                    tmem_ld16_issue(tbase + u * 16, ra);
                    if (GATED) tmem_ld16_issue(tbase + u * 16 + BN, g);
                    uint32_t keep = 0xffffu;
                    if (mask_on && mrow) {
                        keep = 0u;
                        const int s = ep.expert_size;
                        int ee = e, l = lo;
                        while (l < 16) {
                            if ((ee >> 5) != widx) {
                                widx = ee >> 5;
                                word = __ldg(mrow + widx);
                            }
                            const int hi = l + s;
                            if ((word >> (ee & 31)) & 1u) {
                                const int a = l < 0 ? 0 : l, b2 = hi > 16 ? 16 : hi;
                                keep |= ((1u << b2) - 1u) & ~((1u << a) - 1u);
                            }
                            l = hi;
                            ++ee;
                        }
                        // advance to the expert that owns the first column of the next unit
                        lo -= 16;
                        while (lo + s <= 0) { lo += s; ++e; }
                    }
                    tmem_ld_wait();
                    epilogue_16_slow<EPI, ACT, GATED>(ra, g, bias_g, out_p, row, M, col0, N, keep);
                }
            }
            // all of this warp's TMEM reads of the buffer are complete: hand it back to the MMA warp
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bar_acc_empty[buf]));

        }
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS) : "memory");
}

// ------------------------------------------------------------------------------------------ host side

// Band height (in row tiles) for the tile walk, 0 = plain row-major.  Row-major order re-reads B once per wave of
// CTAs, which is free while B stays in L2 (126 MB) beside the streaming A; only a large B (Llama-sized weights) needs
// bands.  The band is sized so that its rows of A take about 32 MB (measured best on the Llama-shaped layer: 32 row
// tiles of 1 MB, 1050 us against 1427 us for the up projection).
int band_rows_for(int M, int N, int K, int tile_m, bool gated)
{
    (void)M;
    const double b_bytes = 2.0 * N * K * (gated ? 2 : 1);
    if (b_bytes < 48e6) return 0;
    const char *e = getenv("D2D_GEMM_BAND");
    if (e) return atoi(e);
    int band = (int)(32e6 / (2.0 * tile_m * K) + 0.5);
    return band < 16 ? 16 : band;                           // shorter bands stream B too often (16 .. 32 measured alike)
}

// cudaFuncAttributeMaxDynamicSharedMemorySize is a per-device attribute: set it once per (kernel, device).
template <typename K> bool ensure_smem_attr(K kern, size_t smem, bool (&done)[64])
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
    if (!__atomic_load_n(&done[dev], __ATOMIC_ACQUIRE)) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return false;
        __atomic_store_n(&done[dev], true, __ATOMIC_RELEASE);
    }
    return true;
}

template <int BN, int EPI, int ACT, bool GATED>
d2d_status launch(const d2d_gemm_args &g, cudaStream_t st)
{
    constexpr int STAGE_BYTES = BM * BK * 2 + (GATED ? 2 : 1) * BN * BK * 2;
    constexpr int STAGES = (200 * 1024) / STAGE_BYTES > 8 ? 8 : (200 * 1024) / STAGE_BYTES;   // 200 KB of operand stages (+ 24 KB bias cache)
    constexpr size_t SMEM = (size_t)STAGES * STAGE_BYTES + 1024 + (size_t)BIAS_CACHE_ELEMS * 4;
    CUtensorMap ta, tb, tb2;
    const bool gate_cat = GATED && g.b_cat != nullptr && g.b_cat_block == BN;
    const int batch = g.batch > 1 ? g.batch : 1;
    if (batch > 1 && (GATED || g.K % BK != 0)) return D2D_ERR_UNSUPPORTED;
    if (!d2d_tc_make_map(&ta, g.a, g.M, g.K * batch, BM)) return D2D_ERR_CUDA;
    if (gate_cat) {
        if (!d2d_tc_make_map(&tb, g.b_cat, 2 * BN * d2d_cdiv(g.N, BN), g.K, 2 * BN)) return D2D_ERR_CUDA;
        tb2 = tb;
    } else {
        if (!d2d_tc_make_map(&tb, g.b, g.N * batch, g.K, BN)) return D2D_ERR_CUDA;
        if (GATED) {
            if (!d2d_tc_make_map(&tb2, g.b_gate, g.N, g.K, BN)) return D2D_ERR_CUDA;
        } else {
            tb2 = tb;
        }
    }
    auto kern = gemm_tc_kernel<BN, STAGES, EPI, ACT, GATED>;
    static bool attr_set[64] = {};
    if (!ensure_smem_attr(kern, SMEM, attr_set)) return D2D_ERR_CUDA;
    const int es = g.expert_size > 0 ? g.expert_size : 1;
    EpiParams ep{(const __nv_bfloat16 *)g.bias, g.out, g.mask, g.mask_words, es, g.status,
                 (uint32_t)((0x100000000ull + (unsigned long long)es - 1) / (unsigned long long)es),
                 g.tile_counter, (g.pdl_late_wait && !g.n_sel && d2d_tc_pdl_enabled()) ? 1 : 0, gate_cat ? 1 : 0,
                 band_rows_for(g.M, g.N, g.K, BM, GATED), batch, g.n_sel, g.n_sel_max,
                 (g.test_skip_load && !g.tile_counter && !g.pdl_late_wait && !g.n_sel) ? 1 : 0};
    const int k_splits = g.k_splits > 1 ? g.k_splits : 1;
    const int tiles = d2d_cdiv(g.N, BN) * d2d_cdiv(g.M, BM) * k_splits * batch;
    const int workers = d2d_tc_sm_count();
    const int grid = tiles < workers ? tiles : workers;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(NTHREADS_V2, 1, 1);
    cfg.dynamicSmemBytes = SMEM;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    // the kernel's prologue may overlap the tail of the previous kernel in the stream (see griddepcontrol.wait in the kernel)
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = d2d_tc_pdl_enabled() ? 1 : 0;
    const cudaError_t err = cudaLaunchKernelEx(&cfg, kern, ta, tb, tb2, ep, g.M, g.N, g.K, k_splits);
    D2D_LAUNCHED(1);
    return err == cudaSuccess && cudaGetLastError() == cudaSuccess ? D2D_OK : D2D_ERR_CUDA;
}

// Tile width with the least modelled time: rounds over the SMs x the time of one 64-deep k-block of a 128 x bn tile.
// That time is not proportional to bn: every k-block brings 16 KB of A and bn / 8 KB of B into the SM, and the SM's
// path from L2 is what a 128-row tile saturates, so a narrow tile pays almost as much as a wide one for fewer columns.
// Measured on B200 (K = 11008, T = 4096 and 8192): 0.40 us per k-block at bn = 256, 0.31 us at bn = 128, i.e. about
// 0.13 us + 0.7 ns per row of A and B staged.  Wider tiles win ties.
int pick_bn(int M, int N, int tile_m, int workers, const int *cands, int n_cands, int batch = 1)
{
    int best = cands[0];
    double best_cost = 1e300;
    for (int i = 0; i < n_cands; ++i) {
        const int bn = cands[i];
        const long tiles = (long)d2d_cdiv(N, bn) * d2d_cdiv(M, tile_m) * batch;
        const long rounds = (tiles + workers - 1) / workers;
        const double cost = (double)rounds * (0.13 + 0.0007 * (double)(tile_m + bn));
        if (cost < best_cost - 1e-9) { best_cost = cost; best = bn; }
    }
    return best;
}

template <int EPI, int ACT, bool GATED>
d2d_status launch_bn(const d2d_gemm_args &g, cudaStream_t st)
{
    if (GATED) return launch<128, EPI, ACT, true>(g, st);
    const int cands[4] = {256, 192, 128, 64};
    switch (pick_bn(g.M, g.N, BM, d2d_tc_sm_count(), cands, 4, g.batch > 1 ? g.batch : 1)) {
    case 256: return launch<256, EPI, ACT, false>(g, st);
    case 192: return launch<192, EPI, ACT, false>(g, st);
    case 128: return launch<128, EPI, ACT, false>(g, st);
    default: return launch<64, EPI, ACT, false>(g, st);
    }
}

template <bool GATED>
d2d_status launch_up(const d2d_gemm_args &g, cudaStream_t st)
{
    switch (g.act) {
    case D2D_ACT_RELU: return launch_bn<D2D_EPI_UP_MASKED, D2D_ACT_RELU, GATED>(g, st);
    case D2D_ACT_GELU_ERF: return launch_bn<D2D_EPI_UP_MASKED, D2D_ACT_GELU_ERF, GATED>(g, st);
    case D2D_ACT_GELU_TANH: return launch_bn<D2D_EPI_UP_MASKED, D2D_ACT_GELU_TANH, GATED>(g, st);
    case D2D_ACT_SILU: return launch_bn<D2D_EPI_UP_MASKED, D2D_ACT_SILU, GATED>(g, st);
    }
    return D2D_ERR_INVALID_ARG;
}

}  // namespace

// y = bf16(partial + bias) after a split-K GEMM; `batch` problems back to back ([batch, M, N] sums, [batch, N] bias)
__global__ void __launch_bounds__(256)
splitk_finalize_kernel(const float *__restrict__ partial, const __nv_bfloat16 *__restrict__ bias, __nv_bfloat16 *__restrict__ out,
                       int M, int N, int batch)
{
    const size_t per = (size_t)M * N, total = per * batch;
    for (size_t i = ((size_t)blockIdx.x * 256 + threadIdx.x) * 4; i < total; i += (size_t)gridDim.x * 1024) {
        const float4 v = __ldcg(reinterpret_cast<const float4 *>(partial + i));
        const int c = (int)(i / per) * N + (int)(i % N);
        const float o[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int q = 0; q < 4; ++q) out[i + q] = __float2bfloat16_rn(o[q] + (bias ? __bfloat162float(bias[c + q]) : 0.0f));
    }
}

namespace {

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

}  // namespace

bool d2d_tc_make_map(CUtensorMap *map, const void *base, int rows, int cols, int box_rows)
{
    encode_tiled_fn enc = get_encode();
    if (!enc) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {64u, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int d2d_tc_sm_count()
{
    static int cached = 0;
    if (cached == 0) {
        int dev = 0, n = 0;
        if (cudaGetDevice(&dev) == cudaSuccess &&
            cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0)
            cached = n;
        else
            return 148;
    }
    return cached;
}

// D2D_GEMM_PDL=0 launches every GEMM fully serialised (no programmatic dependent launch)
bool d2d_tc_pdl_enabled()
{
    static const bool on = [] {
        const char *e = getenv("D2D_GEMM_PDL");
        return !(e && e[0] == '0');
    }();
    return on;
}

bool d2d_gemm_tc_available() { return get_encode() != nullptr; }

int d2d_gemm_tc_splits(int M, int N, int K, int batch)
{
    // only problems whose 128 x 64 output tiles would occupy less than half of the SMs (a few hundred tokens at most)
    if (N & 3) return 1;
    const int tiles = d2d_cdiv(M, BM) * d2d_cdiv(N, 64) * (batch > 1 ? batch : 1);
    const int nkb = d2d_cdiv(K, BK);
    int splits = d2d_tc_sm_count() / (tiles > 0 ? tiles : 1);
    if (splits > nkb / 2) splits = nkb / 2;          // at least two k-blocks per slice
    return splits >= 2 ? splits : 1;
}

d2d_status d2d_gemm_tc(const d2d_gemm_args &g, cudaStream_t st)
{
    if (g.M <= 0 || g.N <= 0 || g.K <= 0) return D2D_OK;
    if (g.K % 8) return D2D_ERR_UNSUPPORTED;
    switch (g.epilogue) {
    case D2D_EPI_RELU_BF16: return launch_bn<D2D_EPI_RELU_BF16, 0, false>(g, st);
    case D2D_EPI_ABS_F32: return launch_bn<D2D_EPI_ABS_F32, 0, false>(g, st);
    case D2D_EPI_BIAS_BF16:
        if (g.k_splits > 1 && g.partial) {
            const int batch = g.batch > 1 ? g.batch : 1;
            if (cudaMemsetAsync(g.partial, 0, (size_t)batch * g.M * g.N * sizeof(float), st) != cudaSuccess) return D2D_ERR_CUDA;
            d2d_gemm_args p = g;
            p.epilogue = D2D_EPI_PARTIAL_F32;
            p.bias = nullptr;
            p.out = g.partial;
            const d2d_status rc = launch<64, D2D_EPI_PARTIAL_F32, 0, false>(p, st);
            if (rc != D2D_OK) return rc;
            const int blocks = d2d_cdiv(batch * g.M * g.N, 1024);
            splitk_finalize_kernel<<<blocks < 148 ? blocks : 148, 256, 0, st>>>(g.partial, (const __nv_bfloat16 *)g.bias,
                                                                                 (__nv_bfloat16 *)g.out, g.M, g.N, batch);
            D2D_LAUNCHED(1);
            return cudaGetLastError() == cudaSuccess ? D2D_OK : D2D_ERR_CUDA;
        }
        return launch_bn<D2D_EPI_BIAS_BF16, 0, false>(g, st);
    case D2D_EPI_UP_MASKED: return g.b_gate ? launch_up<true>(g, st) : launch_up<false>(g, st);
    }
    return D2D_ERR_INVALID_ARG;
}
