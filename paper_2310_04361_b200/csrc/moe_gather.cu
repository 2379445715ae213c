// Gathered, grouped expert up projection (Sec. 3.4, Listing 1: tokens are bucketed by expert and each expert runs
// a contraction over its own tokens only), bf16 on the tcgen05 tensor cores of sm_100a.
//
// A work unit is a GROUP of g adjacent experts (g * s = gs columns of W1, 64 .. 256 of them, so that one MMA is wide
// enough to run the tensor pipe at its full rate) and the tokens that keep at least one expert of the group.  Those
// token rows are gathered into the swizzled A stages, multiplied with the group's contiguous W1 (and W_gate) rows,
// and the epilogue applies bias, activation and the per-(token, expert) selection bits and scatters the gs hidden
// activations of each row to H[token, group columns].  Rows of H that no expert of the group keeps are written as
// zeros by the scheduler warp, so H is complete and the dense down projection can follow.  Executed work is
// proportional to the number of (token, group) pairs, not to T * d_ff.
//
// One persistent CTA per SM, 14 warps:
//   warp 0      scheduler: draws 256-token sub-chunks of a group from per-group device counters (work stealing at
//               256-token granularity, so the CTAs finish together whatever the distribution of tokens over experts),
//               compacts the tokens that keep the group with ballots into a row FIFO in shared memory, writes the zero
//               rows, and emits 128-row tiles (rows left over are carried into the next sub-chunk of the same group;
//               only the last tile of a group visit is ragged)
//   warp 1      allocates TMEM, issues tcgen05.mma (M = 128, N = gs or 2 gs for gated layers), two accumulators
//   warps 2-5   gather: thread (row, 16-byte chunk) copies x rows with cp.async into the 128-byte-swizzled K-major
//               layout the MMA descriptors expect; a group of copies is made visible to the tensor-core (async) proxy
//               with fence.proxy.async before the stage's barrier is signalled.  Warp 2 also requests the W1 tiles
//               (plain per-CTA TMA loads).
//   warps 6-13  epilogue: tcgen05.ld, bias, activation, selection bits, 32-byte stores to the token's row of H
// Every wait is bounded (status D2D_ERR_TIMEOUT), all roles meet at the final barrier, TMEM is freed.
#include "moe_gather.cuh"
#include "tc_common.cuh"

namespace {

using namespace d2d_tc;

constexpr int BM = 128, BK = 64, UMMA_K = 16;
constexpr int A_BYTES = BM * BK * 2;
constexpr int SUB = 256;                 // tokens per scheduler draw
constexpr int TR = 4;                    // tile descriptors in flight
constexpr int FIFO_CAP = 2048;           // row entries; in use at any time: TR * 128 emitted + 127 pending + SUB new
constexpr int MAX_STAGES = 8;
constexpr int WARP_SCHED = 0, WARP_MMA = 1, WARP_GATHER0 = 2, N_GATHER_WARPS = 4, WARP_EPI0 = 6, N_EPI_WARPS = 8;
constexpr int NTHREADS = 32 * (WARP_EPI0 + N_EPI_WARPS);

struct GatherParams {
    const __nv_bfloat16 *x;          // [T, d]
    const uint32_t *mask;            // [T, W]
    const __nv_bfloat16 *b1;         // [d_ff] or NULL
    __nv_bfloat16 *H;                // [T, d_ff]
    int32_t *status;
    int *ctr;                        // [n_groups] sub-chunk counters + [1] exit ticket, zero at launch, reset by the last CTA
    const int32_t *n_sel;            // selected (token, expert) pairs of this batch, or NULL
    long long n_sel_max;             // the kernel does nothing when *n_sel > n_sel_max (the masked dense path runs instead)
    int T, d, d_ff, W;
    int g, s, gs, n_groups;          // experts per group, expert size, g * s, E / g
    uint32_t inv_s;                  // ceil(2^32 / s)
    int stages, stage_bytes, lag;
};

struct TileDesc {
    int start, n_rows, group;
};

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, uint32_t src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_lag(int lag)
{
    switch (lag) {
    case 0: asm volatile("cp.async.wait_group 0;" ::: "memory"); break;
    case 1: asm volatile("cp.async.wait_group 1;" ::: "memory"); break;
    case 2: asm volatile("cp.async.wait_group 2;" ::: "memory"); break;
    case 3: asm volatile("cp.async.wait_group 3;" ::: "memory"); break;
    case 4: asm volatile("cp.async.wait_group 4;" ::: "memory"); break;
    default: asm volatile("cp.async.wait_group 5;" ::: "memory"); break;
    }
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__host__ __device__ constexpr int pow2_cols(int v) { return v <= 32 ? 32 : v <= 64 ? 64 : v <= 128 ? 128 : 256; }

template <int ACT, bool GATED>
__global__ void __launch_bounds__(NTHREADS, 1)
moe_gather_up_kernel(const __grid_constant__ CUtensorMap tm_w1, const __grid_constant__ CUtensorMap tm_wg, const GatherParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint32_t *fifo = reinterpret_cast<uint32_t *>(smem + (size_t)p.stages * p.stage_bytes);     // [FIFO_CAP] token | bits << 24
    int *zlist = reinterpret_cast<int *>(fifo + FIFO_CAP);                                       // [SUB] tokens whose row of the group is zero
    __shared__ uint64_t bar_full[MAX_STAGES], bar_empty[MAX_STAGES], bar_acc_full[2], bar_acc_empty[2], tile_full[TR], tile_empty[TR];
    __shared__ TileDesc tdesc[TR];
    __shared__ uint32_t tmem_base_holder;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nkb = (p.d + BK - 1) / BK;
    const int n_mma = GATED ? 2 * p.gs : p.gs;              // columns of one MMA = accumulator columns of a tile
    const uint32_t buf_cols = (uint32_t)pow2_cols(n_mma);
    const uint32_t tmem_cols = 2u * buf_cols < 32u ? 32u : 2u * buf_cols;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1 + N_GATHER_WARPS);     // the W1 request (with its byte count) + one arrival per gather warp
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&bar_acc_full[b]), 1);
            mbar_init(smem_u32(&bar_acc_empty[b]), N_EPI_WARPS);
        }
        for (int t = 0; t < TR; ++t) {
            mbar_init(smem_u32(&tile_full[t]), 1);
            mbar_init(smem_u32(&tile_empty[t]), N_GATHER_WARPS + 1 + N_EPI_WARPS);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == WARP_MMA) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_holder)), "r"(tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_holder;
    // everything above overlaps the tail of the previous kernel of the stream; the mask (and x) may be its output
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // density-adaptive dispatch: above the crossover the masked dense kernel, launched next to this one, does the work
    const bool run = p.n_sel == nullptr || (long long)__ldcg(p.n_sel) <= p.n_sel_max;

    if (run && warp == WARP_SCHED) {
        // ------------------------------------------------------------------ scheduler
        const int Ng = p.n_groups, n_sub = (p.T + SUB - 1) / SUB;
        const uint32_t lower = (1u << lane) - 1u;
        const uint32_t gm = (1u << p.g) - 1u;                 // g <= 8
        const int ppr = p.gs >> 3;                            // 16-byte pieces per zero row
        int G = (int)(((long long)blockIdx.x * Ng) / (long long)gridDim.x);
        uint32_t head = 0, emitted = 0, tile_seq = 0;
        bool ok = true;
        auto emit = [&](uint32_t start, int n_rows, int group) -> bool {
            const uint32_t sl = tile_seq % TR, use = tile_seq / TR;
            if (!mbar_wait_warp(smem_u32(&tile_empty[sl]), (use & 1u) ^ 1u, p.status)) return false;
            __syncwarp();                                     // the FIFO entries written by all lanes are ordered before the arrival
            if (lane == 0) {
                tdesc[sl].start = (int)start;
                tdesc[sl].n_rows = n_rows;
                tdesc[sl].group = group;
                mbar_arrive(smem_u32(&tile_full[sl]));
            }
            ++tile_seq;
            return true;
        };
        for (int visited = 0; visited < Ng && ok;) {
            int c = 0;
            if (lane == 0) c = atomicAdd(p.ctr + G, 1);
            c = __shfl_sync(0xffffffffu, c, 0);
            if (c >= n_sub) {
                // this group has no sub-chunk left: flush the rows carried so far as a ragged tile and move on
                if (head != emitted) {
                    ok = emit(emitted % FIFO_CAP, (int)(head - emitted), G);
                    emitted = head;
                }
                G = G + 1 == Ng ? 0 : G + 1;
                ++visited;
                continue;
            }
            const int t0 = c * SUB;
            const int e0 = G * p.g, w = e0 >> 5, sh = e0 & 31;
            uint32_t bits[SUB / 32];
#pragma unroll
            for (int j = 0; j < SUB / 32; ++j) {
                const int t = t0 + j * 32 + lane;
                bits[j] = t < p.T ? ((__ldg(p.mask + (size_t)t * p.W + w) >> sh) & gm) : 0u;
            }
            int nz = 0;
#pragma unroll
            for (int j = 0; j < SUB / 32; ++j) {
                const int t = t0 + j * 32 + lane;
                const bool keep = bits[j] != 0u, zero = !keep && t < p.T;
                const uint32_t bk = __ballot_sync(0xffffffffu, keep), bz = __ballot_sync(0xffffffffu, zero);
                if (keep) fifo[(head + __popc(bk & lower)) % FIFO_CAP] = (uint32_t)t | (bits[j] << 24);
                if (zero) zlist[nz + __popc(bz & lower)] = t;
                head += __popc(bk);
                nz += __popc(bz);
            }
            __syncwarp();
            while (head - emitted >= (uint32_t)BM && ok) {
                ok = emit(emitted % FIFO_CAP, BM, G);
                emitted += BM;
            }
            // rows of H that no expert of this group keeps are zero (the dense down projection reads all of H)
            const int pieces = nz * ppr;
            for (int i = lane; i < pieces; i += 32) {
                const int r = i / ppr, q = i - r * ppr;
                __nv_bfloat16 *o = p.H + (size_t)zlist[r] * p.d_ff + (size_t)G * p.gs + q * 8;
                *reinterpret_cast<uint4 *>(o) = make_uint4(0u, 0u, 0u, 0u);
            }
            __syncwarp();                                     // zlist is rewritten by the next draw
        }
        emit(0u, -1, 0);                                      // end of the tile stream
        // the CTA whose scheduler finishes last leaves the counters at zero for the next launch
        if (lane == 0) {
            __threadfence();
            const int done = atomicAdd(p.ctr + Ng, 1);
            if (done == (int)gridDim.x - 1) {
                for (int i = 0; i <= Ng; ++i) p.ctr[i] = 0;
                __threadfence();
            }
        }
    } else if (run && warp == WARP_MMA) {
        // ------------------------------------------------------------------ MMA issuer (whole warp walks, one lane issues)
        const uint32_t idesc = instr_desc_bf16(BM, n_mma);
        uint32_t it = 0;
        bool ok = true;
        for (uint32_t ti = 0; ok; ++ti) {
            const uint32_t sl = ti % TR;
            ok = mbar_wait_warp(smem_u32(&tile_full[sl]), (ti / TR) & 1u, p.status);
            if (!ok) break;
            const int n_rows = tdesc[sl].n_rows;
            __syncwarp();
            if (n_rows < 0) break;
            if (elect_one()) mbar_arrive(smem_u32(&tile_empty[sl]));
            const uint32_t buf = ti & 1u, use = ti >> 1;
            ok = mbar_wait_warp(smem_u32(&bar_acc_empty[buf]), (use & 1u) ^ 1u, p.status);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t acc = tmem_base + buf * buf_cols;
            for (int kb = 0; kb < nkb; ++kb, ++it) {
                const uint32_t s = it % (uint32_t)p.stages, round = it / (uint32_t)p.stages;
                ok = mbar_wait_warp(smem_u32(&bar_full[s]), round & 1u, p.status);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t a_addr = smem_u32(smem + (size_t)s * p.stage_bytes);
                const uint64_t da = smem_desc_sw128(a_addr), db = smem_desc_sw128(a_addr + A_BYTES);
                if (elect_one()) {
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k) {
                        const uint64_t koff = (uint64_t)((k * UMMA_K * 2) >> 4);
                        umma_bf16(acc, da + koff, db + koff, idesc, (kb > 0 || k > 0) ? 1u : 0u);
                    }
                    umma_commit(smem_u32(&bar_empty[s]));
                }
                __syncwarp();
            }
            if (!ok) break;
            if (elect_one()) umma_commit(smem_u32(&bar_acc_full[buf]));
            __syncwarp();
        }
    } else if (run && warp >= WARP_GATHER0 && warp < WARP_EPI0) {
        // ------------------------------------------------------------------ gather warps: x rows -> swizzled A stages
        const int gw = warp - WARP_GATHER0, tid_g = gw * 32 + lane;
        const int chunk = tid_g & 7, rbase = tid_g >> 3;      // this thread copies chunk `chunk` of rows rbase + 16 j
        const uint32_t swz = (uint32_t)(((chunk ^ (rbase & 7)) << 4) + (rbase & 7) * 128 + (rbase >> 3) * 1024);
        uint32_t it = 0, signaled = 0;
        bool ok = true;
        auto drain = [&]() {
            cp_async_wait_lag(0);
            fence_async_smem();
            __syncwarp();
            for (; signaled < it; ++signaled)
                if (lane == 0) mbar_arrive(smem_u32(&bar_full[signaled % (uint32_t)p.stages]));
        };
        for (uint32_t ti = 0; ok; ++ti) {
            const uint32_t sl = ti % TR, par = (ti / TR) & 1u;
            if (!mbar_test(smem_u32(&tile_full[sl]), par)) drain();       // nothing to overlap with: release what is in flight
            ok = mbar_wait_warp(smem_u32(&tile_full[sl]), par, p.status);
            if (!ok) break;
            const int start = tdesc[sl].start, n_rows = tdesc[sl].n_rows, G = tdesc[sl].group;
            if (n_rows < 0) break;
            const __nv_bfloat16 *src[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                int r = rbase + 16 * j;
                r = r < n_rows ? r : n_rows - 1;              // rows past the end of a ragged tile repeat its last row (never stored)
                const uint32_t e = fifo[(uint32_t)(start + r) % FIFO_CAP];
                src[j] = p.x + (size_t)(e & 0xffffffu) * p.d + chunk * 8;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&tile_empty[sl]));
            for (int kb = 0; kb < nkb; ++kb) {
                const uint32_t s = it % (uint32_t)p.stages, round = it / (uint32_t)p.stages;
                ok = mbar_wait_warp(smem_u32(&bar_empty[s]), (round & 1u) ^ 1u, p.status);
                if (!ok) break;
                const uint32_t stage = smem_u32(smem + (size_t)s * p.stage_bytes);
                if (gw == 0 && elect_one()) {
                    const uint32_t full = smem_u32(&bar_full[s]);
                    mbar_expect_tx(full, (uint32_t)(p.stage_bytes - A_BYTES));
                    tma_load_2d(stage + A_BYTES, &tm_w1, kb * BK, G * p.gs, full);
                    if (GATED) tma_load_2d(stage + A_BYTES + p.gs * 128, &tm_wg, kb * BK, G * p.gs, full);
                }
                const uint32_t nbytes = kb * BK + chunk * 8 < p.d ? 16u : 0u;      // zero fill past K
#pragma unroll
                for (int j = 0; j < 8; ++j) cp_async16(stage + swz + (uint32_t)j * 2048u, nbytes ? src[j] + kb * BK : p.x, nbytes);
                cp_async_commit();
                ++it;
                if (it - signaled > (uint32_t)p.lag) {
                    cp_async_wait_lag(p.lag);
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&bar_full[signaled % (uint32_t)p.stages]));
                    ++signaled;
                }
            }
        }
        drain();
    } else if (run && warp >= WARP_EPI0) {
        // ------------------------------------------------------------------ epilogue
        const int ew = warp - WARP_EPI0, quad = warp & 3, half = ew >> 2;
        const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
        const int n_units = p.gs >> 4;
        const bool halves = (p.s & 7) == 0;                   // every 8-column half of a unit belongs to one expert
        const bool wide = (p.d_ff & 15) == 0 && (reinterpret_cast<uintptr_t>(p.H) & 31) == 0;
        bool ok = true;
        for (uint32_t ti = 0; ok; ++ti) {
            const uint32_t sl = ti % TR;
            ok = mbar_wait_warp(smem_u32(&tile_full[sl]), (ti / TR) & 1u, p.status);
            if (!ok) break;
            const int start = tdesc[sl].start, n_rows = tdesc[sl].n_rows, G = tdesc[sl].group;
            if (n_rows < 0) break;
            const int r = quad * 32 + lane;
            const bool valid = r < n_rows;
            const uint32_t e = valid ? fifo[(uint32_t)(start + r) % FIFO_CAP] : 0u;
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&tile_empty[sl]));
            const uint32_t bits = e >> 24;
            __nv_bfloat16 *orow = p.H + (size_t)(e & 0xffffffu) * p.d_ff + (size_t)G * p.gs;
            const __nv_bfloat16 *brow = p.b1 ? p.b1 + (size_t)G * p.gs : nullptr;
            const uint32_t buf = ti & 1u, use = ti >> 1;
            ok = mbar_wait_warp(smem_u32(&bar_acc_full[buf]), use & 1u, p.status);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t tbase = tmem_base + buf * buf_cols + lane_base;
            for (int u = half; u < n_units; u += 2) {
                const int col0 = u * 16;
                uint32_t ra[16], ga[GATED ? 16 : 1];
                tmem_ld16_issue(tbase + (uint32_t)col0, ra);
                if (GATED) tmem_ld16_issue(tbase + (uint32_t)(p.gs + col0), reinterpret_cast<uint32_t (&)[16]>(ga));
                float bias[16];
                if (brow) {
                    float b8[8];
                    d2d_load8(brow + col0, b8);
#pragma unroll
                    for (int q = 0; q < 8; ++q) bias[q] = b8[q];
                    d2d_load8(brow + col0 + 8, b8);
#pragma unroll
                    for (int q = 0; q < 8; ++q) bias[8 + q] = b8[q];
                } else {
#pragma unroll
                    for (int q = 0; q < 16; ++q) bias[q] = 0.0f;
                }
                uint32_t keep;
                if (halves) {
                    const uint32_t e_lo = __umulhi((uint32_t)col0, p.inv_s), e_hi = __umulhi((uint32_t)(col0 + 8), p.inv_s);
                    keep = ((bits >> e_lo) & 1u ? 0x00ffu : 0u) | ((bits >> e_hi) & 1u ? 0xff00u : 0u);
                } else {
                    keep = 0u;
#pragma unroll
                    for (int j = 0; j < 16; ++j) keep |= ((bits >> __umulhi((uint32_t)(col0 + j), p.inv_s)) & 1u) << j;
                }
                tmem_ld_wait();
                uint32_t pk[8];
#pragma unroll
                for (int j = 0; j < 16; j += 2) {
                    const uint64_t z = add2(pack2(__uint_as_float(ra[j]), __uint_as_float(ra[j + 1])), pack2(bias[j], bias[j + 1]));
                    const uint64_t h = GATED ? mul2(fast_act2<ACT>(pack2(__uint_as_float(ga[GATED ? j : 0]), __uint_as_float(ga[GATED ? j + 1 : 0]))), z)
                                             : fast_act2<ACT>(z);
                    float v0, v1;
                    unpack2(h, v0, v1);
                    const __nv_bfloat162 t2 = __floats2bfloat162_rn(v0, v1);
                    uint32_t wv = *reinterpret_cast<const uint32_t *>(&t2);
                    // an expert the token did not keep contributes zeros (also when its pre-activations are not finite)
                    wv = (keep >> j) & 1u ? wv : (wv & 0xffff0000u);
                    wv = (keep >> (j + 1)) & 1u ? wv : (wv & 0x0000ffffu);
                    pk[j >> 1] = wv;
                }
                if (valid) {
                    __nv_bfloat16 *o = orow + col0;
                    if (wide) {
                        asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(o), "r"(pk[0]), "r"(pk[1]), "r"(pk[2]),
                                     "r"(pk[3]), "r"(pk[4]), "r"(pk[5]), "r"(pk[6]), "r"(pk[7]) : "memory");
                    } else {
                        *reinterpret_cast<uint4 *>(o) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                        *reinterpret_cast<uint4 *>(o + 8) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
                    }
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bar_acc_empty[buf]));
        }
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == WARP_MMA)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
}

template <int ACT, bool GATED>
d2d_status launch(const d2d_gather_args &a, cudaStream_t st)
{
    const int gs = a.g * a.s;
    const int b_rows = GATED ? 2 * gs : gs;
    GatherParams p = {};
    p.x = (const __nv_bfloat16 *)a.x; p.mask = a.mask; p.b1 = (const __nv_bfloat16 *)a.b1; p.H = (__nv_bfloat16 *)a.H;
    p.status = a.status; p.ctr = a.ctr; p.n_sel = a.n_sel; p.n_sel_max = a.n_sel_max;
    p.T = a.T; p.d = a.d; p.d_ff = a.d_ff; p.W = (a.n_experts + 31) / 32;
    p.g = a.g; p.s = a.s; p.gs = gs; p.n_groups = a.n_experts / a.g;
    p.inv_s = (uint32_t)((0x100000000ull + (unsigned long long)a.s - 1) / (unsigned long long)a.s);
    p.stage_bytes = A_BYTES + b_rows * 128;
    int stages = (192 * 1024) / p.stage_bytes;
    p.stages = stages > MAX_STAGES ? MAX_STAGES : stages;
    p.lag = p.stages - 2 > 4 ? 4 : p.stages - 2;
    const size_t smem = (size_t)p.stages * p.stage_bytes + FIFO_CAP * 4 + SUB * 4 + 1024;      // at most 192 + 8 + 1 + 1 KB
    if (smem > 208 * 1024) return D2D_ERR_UNSUPPORTED;
    CUtensorMap tw1, twg;
    if (!d2d_tc_make_map(&tw1, a.w1, a.d_ff, a.d, gs)) return D2D_ERR_CUDA;
    if (GATED) {
        if (!d2d_tc_make_map(&twg, a.w_gate, a.d_ff, a.d, gs)) return D2D_ERR_CUDA;
    } else {
        twg = tw1;
    }
    auto kern = moe_gather_up_kernel<ACT, GATED>;
    static bool attr_set[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return D2D_ERR_CUDA;
    if (!__atomic_load_n(&attr_set[dev], __ATOMIC_ACQUIRE)) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 208 * 1024) != cudaSuccess) return D2D_ERR_CUDA;
        __atomic_store_n(&attr_set[dev], true, __ATOMIC_RELEASE);
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(d2d_tc_sm_count(), 1, 1);
    cfg.blockDim = dim3(NTHREADS, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = d2d_tc_pdl_enabled() ? 1 : 0;
    const cudaError_t err = cudaLaunchKernelEx(&cfg, kern, tw1, twg, p);
    D2D_LAUNCHED(1);
    return err == cudaSuccess && cudaGetLastError() == cudaSuccess ? D2D_OK : D2D_ERR_CUDA;
}

template <bool GATED>
d2d_status launch_act(const d2d_gather_args &a, cudaStream_t st)
{
    switch (a.act) {
    case D2D_ACT_RELU: return launch<D2D_ACT_RELU, GATED>(a, st);
    case D2D_ACT_GELU_ERF: return launch<D2D_ACT_GELU_ERF, GATED>(a, st);
    case D2D_ACT_GELU_TANH: return launch<D2D_ACT_GELU_TANH, GATED>(a, st);
    case D2D_ACT_SILU: return launch<D2D_ACT_SILU, GATED>(a, st);
    }
    return D2D_ERR_INVALID_ARG;
}

}  // namespace

int d2d_gather_group_for(const d2d_layer_desc &D, int want)
{
    if (D.dtype != D2D_BF16 || D.d % 8 || D.d_ff % 8 || D.expert_size % 8 || !d2d_gemm_tc_available()) return 0;
    const int max_cols = D.gated ? 128 : 256;                 // one MMA holds gs (gated: 2 gs) accumulator columns
    auto fits = [&](int g) {
        const int gs = g * D.expert_size;
        return g >= 1 && g <= 8 && D.n_experts % g == 0 && 32 % g == 0 && gs % 16 == 0 && gs >= 16 && gs <= max_cols;
    };
    if (want > 0) return fits(want) ? want : 0;
    // default: the widest group of at most 128 columns (a full-rate MMA without wasting rows on a larger union)
    for (int g = 8; g >= 1; g >>= 1)
        if (fits(g) && g * D.expert_size <= 128) return g;
    return fits(1) ? 1 : 0;
}

d2d_status d2d_moe_gather_up(const d2d_gather_args &a, cudaStream_t st)
{
    if (a.T <= 0) return D2D_OK;
    if (a.T >= (1 << 24) || a.g < 1 || a.g > 8) return D2D_ERR_UNSUPPORTED;
    return a.w_gate ? launch_act<true>(a, st) : launch_act<false>(a, st);
}
