// Gathered, grouped expert up projection (Sec. 3.4, Listing 1: tokens are bucketed by expert and each expert runs
// a contraction over its own tokens only), bf16 on the tcgen05 tensor cores of sm_100a.
//
// A work unit is a GROUP of g adjacent experts (g * s = gs columns of W1, 64 .. 256 of them, so that one MMA is wide
// enough to run the tensor pipe at its full rate) and the tokens that keep at least one expert of the group.  Those
// token rows are gathered into the swizzled A stages, multiplied with the group's contiguous W1 (and W_gate) rows,
// and the epilogue applies bias, activation and the per-(token, expert) selection bits and scatters the gs hidden
// activations of each row to H[token, group columns].  Cells of H whose (token, group) pair is not kept are NOT
// written: the down projection that follows (moe_down_masked_kernel below) never reads them, it zero-fills those
// pieces of its A operand from the selection mask instead.  Executed work is proportional to the number of
// (token, group) pairs, not to T * d_ff.
//
// One persistent CTA per SM, 14 warps:
//   warp 0      scheduler: draws 256-token sub-chunks of a group from per-group device counters (work stealing at
//               256-token granularity, so the CTAs finish together whatever the distribution of tokens over experts),
//               compacts the tokens that keep the group with ballots into a row FIFO in shared memory and emits 128-row
//               tiles (rows left over are carried into the next sub-chunk of the same group; only the last tile of a
//               group visit is ragged)
//   warp 1      allocates TMEM, issues tcgen05.mma (M = 128, N = gs or 2 gs for gated layers), two accumulators
//   warps 2-5   gather: thread (row, 16-byte chunk) copies x rows with cp.async into the 128-byte-swizzled K-major
//               layout the MMA descriptors expect and lets the copies themselves arrive on the stage's barrier
//               (cp.async.mbarrier.arrive), so the threads never wait for data; the MMA warp executes the
//               generic-to-async proxy fence after it has seen the barrier complete.  Warp 2 also requests the W1
//               tiles (plain per-CTA TMA loads).  Measured alternatives, all slower or equal on B200: a fence in every
//               gather thread after cp.async.wait_group (the threads then wait for data); one warp per stage that
//               copies, waits, fences and signals; eight gather warps; one fence for several k-blocks; four-row TMA
//               gathers (cp.async.bulk.tensor tile::gather4: no fence, but about 80 cycles per 512-byte gather).
//               The stage period stays at about half a microsecond per 128 x 64 tile of gathered rows.
//   warps 6-13  epilogue: tcgen05.ld, bias, activation, selection bits, 32-byte stores to the token's row of H
// Every wait is bounded (status D2D_ERR_TIMEOUT), all roles meet at the final barrier, TMEM is freed.
#include "moe_gather.cuh"
#include "tc_common.cuh"

namespace {

using namespace d2d_tc;

constexpr int BM = 128, BK = 64, UMMA_K = 16;
constexpr int A_BYTES = BM * BK * 2;
constexpr int MAX_SUB = 1024;            // most tokens per scheduler draw (a multiple of 256 chosen per launch, see launch())
constexpr int TR = 4;                    // tile descriptors in flight
constexpr int FIFO_CAP = 2048;           // row entries; in use at any time: TR * 128 emitted + 127 pending + MAX_SUB new
constexpr int MAX_STAGES = 8;
#ifndef D2D_GATHER_WARPS
#define D2D_GATHER_WARPS 4
#endif
constexpr int WARP_SCHED = 0, WARP_MMA = 1, WARP_GATHER0 = 2, N_GATHER_WARPS = D2D_GATHER_WARPS, WARP_EPI0 = WARP_GATHER0 + N_GATHER_WARPS,
              N_EPI_WARPS = 8;
constexpr int ROWS_PER_PASS = N_GATHER_WARPS * 4;      // rows one pass of the gather threads covers (8 threads per row)
constexpr int PASSES = BM / ROWS_PER_PASS;              // rows per gather thread and k-block
constexpr int NTHREADS = 32 * (WARP_EPI0 + N_EPI_WARPS);

struct GatherParams {
    const __nv_bfloat16 *x;          // [T, d]
    const uint32_t *mask;            // [T, W]
    const __nv_bfloat16 *b1;         // [d_ff] or NULL
    __nv_bfloat16 *H;                // [T, d_ff]
    int32_t *status;
    int *ctr;                        // [n_groups] sub-chunk counters + [1] exit ticket, zero at launch, reset by the last CTA
    const int32_t *n_sel;            // selected (token, expert) pairs of this batch, or NULL
    long long n_sel_min, n_sel_max;  // the kernel works only when n_sel_min < *n_sel <= n_sel_max (another path runs otherwise)
    int T, d, d_ff, W;
    int g, s, gs, n_groups;          // experts per group, expert size, g * s, E / g
    uint32_t inv_s;                  // ceil(2^32 / s)
    int stages, stage_bytes;
    int window;                      // groups the CTAs work in at the same time (their weight rows stay in L2)
    int sub;                         // tokens per scheduler draw
    float visit_tiles;               // full tiles a group visit should yield when the density allows it
};

struct TileDesc {
    int start, n_rows, group;
};

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, uint32_t src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
// one arrival on the barrier (counted in its initial count) once all earlier cp.async of this thread have completed
__device__ __forceinline__ void cp_async_arrive(uint32_t bar)
{
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__host__ __device__ constexpr int pow2_cols(int v) { return v <= 32 ? 32 : v <= 64 ? 64 : v <= 128 ? 128 : 256; }

// The MMA warp's work for one tile: nkb k-blocks from the stage ring into the accumulator at `acc`.  The A tiles were
// written by cp.async (generic proxy) and their arrival is observed through the stage's barrier; the proxy fence that
// makes them visible to the tensor core's (async-proxy) reads is executed here, between that observation and the MMAs.
__device__ __forceinline__ bool mma_tile(uint8_t *smem, uint64_t *bar_full, uint64_t *bar_empty, uint64_t *acc_full, uint32_t acc,
                                         uint32_t idesc, int nkb, int stages, int stage_bytes, uint32_t &it, int32_t *status)
{
    for (int kb = 0; kb < nkb; ++kb, ++it) {
        const uint32_t s = it % (uint32_t)stages, round = it / (uint32_t)stages;
        if (!mbar_wait_warp(smem_u32(&bar_full[s]), round & 1u, status)) return false;
        fence_async_smem();
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t a_addr = smem_u32(smem + (size_t)s * stage_bytes);
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
    if (elect_one()) umma_commit(smem_u32(acc_full));
    __syncwarp();
    return true;
}

// The scheduler warp's whole job (see the file header): draws sub-chunks of groups from the device counters, compacts
// the tokens that keep the group into the FIFO, emits tiles through the descriptor ring, ends the stream with a
// sentinel, and lets the CTA that finishes last reset the counters.
__device__ __forceinline__ void run_scheduler(const GatherParams &p, uint32_t *fifo, uint64_t *tile_full, uint64_t *tile_empty,
                                              TileDesc *tdesc, uint32_t *live, int lane)
{
    const int Ng = p.n_groups, SUB = p.sub, n_sub = (p.T + SUB - 1) / SUB;        // SUB is a multiple of 256
    // Groups the CTAs work in at the same time.  The host's value keeps that many groups' weight rows in L2.  When
    // few tokens keep a group, a visit of a CTA to a group should still yield several full tiles (its last tile is
    // ragged and costs as much as a full one), so the CTAs spread over more groups: with gridDim.x / Wn CTAs per
    // group a visit collects about u * T * Wn / gridDim.x rows, u = 1 - (1 - rho)^g the expected kept fraction.
    int Wn = p.window;
    if (p.n_sel) {
        const float rho = fminf((float)__ldcg(p.n_sel) / ((float)p.T * (float)(Ng * p.g)), 1.0f);
        const float u = fmaxf(1.0f - __expf((float)p.g * log1pf(-fminf(rho, 0.999f))), 1e-6f);
        const float need = p.visit_tiles * (float)BM * (float)gridDim.x / (u * (float)p.T);
        const int w = need >= (float)Ng ? Ng : (int)need;
        Wn = w > Wn ? w : Wn;
    }
    const uint32_t lower = (1u << lane) - 1u;
    const uint32_t gm = p.g >= 32 ? 0xffffffffu : (1u << p.g) - 1u;
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
    // Visiting order: the groups are dealt to Wn "lanes" (group G belongs to lane G % Wn).  A CTA first works through
    // its own lane, then through the others, so that at any time the CTAs are busy in about Wn groups whose weight
    // rows stay in L2 while the token rows stream by.  Before it picks its next group a CTA takes a snapshot of all
    // counters (one round trip for the whole warp) and skips the groups that are used up: a counter only grows, so
    // "used up" is final and the walk over the order below never has to go back.
    int j = 0, G = (int)blockIdx.x % Wn;                  // position in the order: lane (blockIdx.x + j) % Wn, group G
    while (ok) {
        for (int base = 0; base < Ng; base += 32) {
            const int gi = base + lane;
            const bool alive = gi < Ng && *(volatile const int *)(p.ctr + gi) < n_sub;
            const uint32_t b = __ballot_sync(0xffffffffu, alive);
            if (lane == 0) live[base >> 5] = b;
        }
        __syncwarp();
        while (j < Wn && !((live[G >> 5] >> (G & 31)) & 1u)) {
            G += Wn;
            if (G >= Ng) {
                ++j;
                G = ((int)blockIdx.x + j) % Wn;
            }
        }
        __syncwarp();                                     // everyone has read the snapshot before it is rewritten
        if (j >= Wn) break;               // every group is used up
        const int e0 = G * p.g, w = e0 >> 5, sh = e0 & 31;
        // Draws of this group, software-pipelined: the counter is bumped one draw ahead, and a draw is walked in
        // pieces of 256 tokens (eight mask words per lane) whose loads are requested one piece ahead of the
        // compaction, so the warp waits for one memory latency per draw, not per piece.
        auto load_piece = [&](int t0, uint32_t (&bits)[8]) {
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const int t = t0 + q * 32 + lane;
                bits[q] = t < p.T ? ((__ldg(p.mask + (size_t)t * p.W + w) >> sh) & gm) : 0u;
            }
        };
        int c = 0;
        if (lane == 0) c = atomicAdd(p.ctr + G, 1);
        c = __shfl_sync(0xffffffffu, c, 0);
        while (c < n_sub && ok) {
            int c_next = 0;
            if (lane == 0) c_next = atomicAdd(p.ctr + G, 1);       // its round trip overlaps this draw
            const int t_end = min((c + 1) * SUB, p.T);
            uint32_t bits[8], bits_next[8];
            load_piece(c * SUB, bits);
            for (int t0 = c * SUB; t0 < t_end && ok; t0 += 256) {
                if (t0 + 256 < t_end) load_piece(t0 + 256, bits_next);
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const bool keep = bits[q] != 0u;
                    const uint32_t bk = __ballot_sync(0xffffffffu, keep);
                    if (keep) fifo[(head + __popc(bk & lower)) % FIFO_CAP] = (uint32_t)(t0 + q * 32 + lane);
                    head += __popc(bk);
                }
                while (head - emitted >= (uint32_t)BM && ok) {
                    ok = emit(emitted % FIFO_CAP, BM, G);
                    emitted += BM;
                }
#pragma unroll
                for (int q = 0; q < 8; ++q) bits[q] = bits_next[q];
            }
            c = __shfl_sync(0xffffffffu, c_next, 0);
        }
        // no sub-chunk of this group is left: the rows carried so far go out as a ragged tile
        if (ok && head != emitted) {
            ok = emit(emitted % FIFO_CAP, (int)(head - emitted), G);
            emitted = head;
        }
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
}

template <int ACT, bool GATED>
__global__ void __launch_bounds__(NTHREADS, 1)
moe_gather_up_kernel(const __grid_constant__ CUtensorMap tm_w1, const __grid_constant__ CUtensorMap tm_wg, const GatherParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint32_t *fifo = reinterpret_cast<uint32_t *>(smem + (size_t)p.stages * p.stage_bytes);     // [FIFO_CAP] token indices
    __shared__ uint64_t bar_full[MAX_STAGES], bar_empty[MAX_STAGES], bar_acc_full[2], bar_acc_empty[2], tile_full[TR], tile_empty[TR];
    __shared__ TileDesc tdesc[TR];
    __shared__ uint32_t tmem_base_holder;
    __shared__ uint32_t live[64];                             // scheduler: groups that still have sub-chunks (one bit each, E <= 2048)

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nkb = (p.d + BK - 1) / BK;
    const int n_mma = GATED ? 2 * p.gs : p.gs;              // columns of one MMA = accumulator columns of a tile
    const uint32_t buf_cols = (uint32_t)pow2_cols(n_mma);
    const uint32_t tmem_cols = 2u * buf_cols < 32u ? 32u : 2u * buf_cols;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            // the W1 request (with its byte count) + one arrival per gather thread, triggered when its copies have landed
            mbar_init(smem_u32(&bar_full[s]), 1 + N_GATHER_WARPS * 32);
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
    const long long n_sel_now = p.n_sel ? (long long)__ldcg(p.n_sel) : 0;
    const bool run = p.n_sel == nullptr || (n_sel_now > p.n_sel_min && n_sel_now <= p.n_sel_max);      // (-1, LLONG_MAX]: always

    if (run && warp == WARP_SCHED) {
        run_scheduler(p, fifo, tile_full, tile_empty, tdesc, live, lane);
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
            ok = mma_tile(smem, bar_full, bar_empty, &bar_acc_full[buf], tmem_base + buf * buf_cols, idesc, nkb, p.stages, p.stage_bytes, it,
                          p.status);
        }
    } else if (run && warp >= WARP_GATHER0 && warp < WARP_EPI0) {
        // ------------------------------------------------------------------ gather warps: x rows -> swizzled A stages
        const int gw = warp - WARP_GATHER0, tid_g = gw * 32 + lane;
        const int chunk = tid_g & 7, rbase = tid_g >> 3;      // this thread copies chunk `chunk` of rows rbase + ROWS_PER_PASS * j
        const uint32_t swz = (uint32_t)(((chunk ^ (rbase & 7)) << 4) + (rbase & 7) * 128 + (rbase >> 3) * 1024);
        uint32_t it = 0;
        bool ok = true;
        for (uint32_t ti = 0; ok; ++ti) {
            const uint32_t sl = ti % TR;
            ok = mbar_wait_warp(smem_u32(&tile_full[sl]), (ti / TR) & 1u, p.status);
            if (!ok) break;
            const int start = tdesc[sl].start, n_rows = tdesc[sl].n_rows, G = tdesc[sl].group;
            if (n_rows < 0) break;
            const __nv_bfloat16 *src[PASSES];
#pragma unroll
            for (int j = 0; j < PASSES; ++j) {
                int r = rbase + ROWS_PER_PASS * j;
                // rows past the end of a ragged tile are zero-filled (no memory traffic) and never stored
                src[j] = r < n_rows ? p.x + (size_t)fifo[(uint32_t)(start + r) % FIFO_CAP] * p.d + chunk * 8 : nullptr;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&tile_empty[sl]));
            for (int kb = 0; kb < nkb; ++kb, ++it) {
                const uint32_t s = it % (uint32_t)p.stages, round = it / (uint32_t)p.stages;
                ok = mbar_wait_warp(smem_u32(&bar_empty[s]), (round & 1u) ^ 1u, p.status);
                if (!ok) break;
                const uint32_t stage = smem_u32(smem + (size_t)s * p.stage_bytes), full = smem_u32(&bar_full[s]);
                if (gw == 0 && elect_one()) {
                    mbar_expect_tx(full, (uint32_t)(p.stage_bytes - A_BYTES));
                    tma_load_2d(stage + A_BYTES, &tm_w1, kb * BK, G * p.gs, full);
                    if (GATED) tma_load_2d(stage + A_BYTES + p.gs * 128, &tm_wg, kb * BK, G * p.gs, full);
                }
                const bool in_k = kb * BK + chunk * 8 < p.d;                       // zero fill past K
#pragma unroll
                for (int j = 0; j < PASSES; ++j) {
                    const bool live_row = in_k && src[j] != nullptr;
                    cp_async16(stage + swz + (uint32_t)(j * ROWS_PER_PASS * 128), live_row ? src[j] + kb * BK : p.x, live_row ? 16u : 0u);
                }
                cp_async_arrive(full);                        // arrives when this thread's copies above have landed
            }
        }
        cp_async_wait_all();                                  // nothing of this thread is in flight when the CTA exits
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
            const uint32_t tok = valid ? fifo[(uint32_t)(start + r) % FIFO_CAP] : 0u;
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&tile_empty[sl]));
            // which experts of the group this token keeps (the load is covered by the wait for the accumulator)
            const int e0 = G * p.g;
            const uint32_t bits = valid ? __ldg(p.mask + (size_t)tok * p.W + (e0 >> 5)) >> (e0 & 31) : 0u;
            __nv_bfloat16 *orow = p.H + (size_t)tok * p.d_ff + (size_t)G * p.gs;
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

// ---------------------------------------------------------------------------------------------------------------
// Down projection after the gathered up projection: y = Hm W2^T + b2, where Hm[t, n] = G[t, n / s] ? H[t, n] : 0.
// The selection is applied while the A operand is staged: a 16-byte piece of a row of H (8 neurons of one expert)
// is copied only if the token keeps that expert and is zero-filled otherwise (cp.async with a source size of 0), so
// cells of H that the gathered kernel never wrote are never read, and the pieces that are skipped cost no L2 traffic.
// The contraction itself is dense (every token of a 128-token tile keeps some expert of every 64-neuron k-block).
// Same roles as above without the scheduler: tiles are (128 tokens) x (bn columns of y), walked round-robin.
struct DownParams {
    const __nv_bfloat16 *H;          // [T, d_ff]
    const uint32_t *mask;            // [T, W]
    const __nv_bfloat16 *b2;         // [d] or NULL
    __nv_bfloat16 *y;                // [T, d]
    int32_t *status;
    const int32_t *n_sel;            // density-adaptive dispatch: work only when n_sel_min < *n_sel <= n_sel_max (NULL: always)
    long long n_sel_min, n_sel_max;
    int T, d, d_ff, W, s;
    uint32_t inv_s;
    int bn, stages, stage_bytes, band;
};

__global__ void __launch_bounds__(NTHREADS, 1)
moe_down_masked_kernel(const __grid_constant__ CUtensorMap tm_w2, const DownParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ uint64_t bar_full[MAX_STAGES], bar_empty[MAX_STAGES], bar_acc_full[2], bar_acc_empty[2];
    __shared__ uint32_t tmem_base_holder;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nkb = (p.d_ff + BK - 1) / BK;
    const int row_tiles = (p.T + BM - 1) / BM, col_tiles = (p.d + p.bn - 1) / p.bn, total = row_tiles * col_tiles;
    const uint32_t buf_cols = (uint32_t)pow2_cols(p.bn);
    const uint32_t tmem_cols = 2u * buf_cols;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1 + N_GATHER_WARPS * 32);
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&bar_acc_full[b]), 1);
            mbar_init(smem_u32(&bar_acc_empty[b]), N_EPI_WARPS);
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
    asm volatile("griddepcontrol.wait;" ::: "memory");       // H is the previous kernel's output
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const long long n_sel_now = p.n_sel ? (long long)__ldcg(p.n_sel) : 0;
    const bool run = p.n_sel == nullptr || (n_sel_now > p.n_sel_min && n_sel_now <= p.n_sel_max);

    // tile index -> (row tile, column tile): row-major, or column by column inside bands of `band` row tiles when W2 is
    // too large to stay in L2 beside the streaming H (the band's rows of H are then re-used from L2 for every column)
    auto coords = [&](int tile, int &r, int &c) {
        if (p.band <= 0) { r = tile / col_tiles; c = tile - r * col_tiles; return; }
        const int per_band = p.band * col_tiles;
        const int b = tile / per_band, idx = tile - b * per_band;
        const int h = row_tiles - b * p.band < p.band ? row_tiles - b * p.band : p.band;
        c = idx / h;
        r = b * p.band + (idx - c * h);
    };

    if (!run) {
        // the masked dense up projection ran: the plain dense down projection, launched next to this kernel, follows it
    } else if (warp == WARP_MMA) {
        const uint32_t idesc = instr_desc_bf16(BM, p.bn);
        uint32_t it = 0, local = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < total && ok; tile += gridDim.x, ++local) {
            const uint32_t buf = local & 1u, use = local >> 1;
            ok = mbar_wait_warp(smem_u32(&bar_acc_empty[buf]), (use & 1u) ^ 1u, p.status);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            ok = mma_tile(smem, bar_full, bar_empty, &bar_acc_full[buf], tmem_base + buf * buf_cols, idesc, nkb, p.stages, p.stage_bytes, it,
                          p.status);
        }
    } else if (warp >= WARP_GATHER0 && warp < WARP_EPI0) {
        const int gw = warp - WARP_GATHER0, tid_g = gw * 32 + lane;
        const int chunk = tid_g & 7, rbase = tid_g >> 3;
        const uint32_t swz = (uint32_t)(((chunk ^ (rbase & 7)) << 4) + (rbase & 7) * 128 + (rbase >> 3) * 1024);
        uint32_t it = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < total && ok; tile += gridDim.x) {
            int tr, tc;
            coords(tile, tr, tc);
            const int m0 = tr * BM, n0 = tc * p.bn;
            uint32_t mw[PASSES];                              // the mask word that holds the current expert, one per row of this thread
            int cur_w = -1;
            for (int kb = 0; kb < nkb; ++kb, ++it) {
                const uint32_t s = it % (uint32_t)p.stages, round = it / (uint32_t)p.stages;
                const int col = kb * BK + chunk * 8;
                const bool in_k = col < p.d_ff;
                const uint32_t e = __umulhi((uint32_t)col, p.inv_s);     // the expert that owns these 8 neurons
                if (in_k && (int)(e >> 5) != cur_w) {
                    cur_w = (int)(e >> 5);
#pragma unroll
                    for (int j = 0; j < PASSES; ++j) {
                        const int t = m0 + rbase + ROWS_PER_PASS * j;
                        mw[j] = t < p.T ? __ldg(p.mask + (size_t)t * p.W + cur_w) : 0u;
                    }
                }
                ok = mbar_wait_warp(smem_u32(&bar_empty[s]), (round & 1u) ^ 1u, p.status);
                if (!ok) break;
                const uint32_t stage = smem_u32(smem + (size_t)s * p.stage_bytes), full = smem_u32(&bar_full[s]);
                if (gw == 0 && elect_one()) {
                    mbar_expect_tx(full, (uint32_t)(p.stage_bytes - A_BYTES));
                    tma_load_2d(stage + A_BYTES, &tm_w2, kb * BK, n0, full);
                }
                const __nv_bfloat16 *src = p.H + (size_t)(m0 + rbase) * p.d_ff + col;
#pragma unroll
                for (int j = 0; j < PASSES; ++j) {
                    const bool keep = in_k && ((mw[j] >> (e & 31u)) & 1u);
                    cp_async16(stage + swz + (uint32_t)(j * ROWS_PER_PASS * 128), keep ? src + (size_t)(ROWS_PER_PASS * j) * p.d_ff : p.H,
                               keep ? 16u : 0u);
                }
                cp_async_arrive(full);
            }
        }
        cp_async_wait_all();
    } else if (warp >= WARP_EPI0) {
        const int ew = warp - WARP_EPI0, quad = warp & 3, half = ew >> 2;
        const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
        const bool wide = (p.d & 15) == 0 && (reinterpret_cast<uintptr_t>(p.y) & 31) == 0;
        uint32_t local = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < total && ok; tile += gridDim.x, ++local) {
            int tr, tc;
            coords(tile, tr, tc);
            const int row = tr * BM + quad * 32 + lane, n0 = tc * p.bn;
            const uint32_t buf = local & 1u, use = local >> 1;
            ok = mbar_wait_warp(smem_u32(&bar_acc_full[buf]), use & 1u, p.status);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t tbase = tmem_base + buf * buf_cols + lane_base;
            const int n_units = p.bn >> 4;
            for (int u = half; u < n_units; u += 2) {
                const int col0 = n0 + u * 16;
                if (col0 >= p.d) break;                         // ragged last column tile (d is a multiple of 16)
                uint32_t ra[16];
                tmem_ld16_issue(tbase + (uint32_t)(u * 16), ra);
                float bias[16];
                if (p.b2) {
                    float b8[8];
                    d2d_load8(p.b2 + col0, b8);
#pragma unroll
                    for (int q = 0; q < 8; ++q) bias[q] = b8[q];
                    d2d_load8(p.b2 + col0 + 8, b8);
#pragma unroll
                    for (int q = 0; q < 8; ++q) bias[8 + q] = b8[q];
                } else {
#pragma unroll
                    for (int q = 0; q < 16; ++q) bias[q] = 0.0f;
                }
                tmem_ld_wait();
                uint32_t pk[8];
#pragma unroll
                for (int j = 0; j < 16; j += 2) {
                    const __nv_bfloat162 t2 = __floats2bfloat162_rn(__uint_as_float(ra[j]) + bias[j], __uint_as_float(ra[j + 1]) + bias[j + 1]);
                    pk[j >> 1] = *reinterpret_cast<const uint32_t *>(&t2);
                }
                if (row < p.T) {
                    __nv_bfloat16 *o = p.y + (size_t)row * p.d + col0;
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

// ---------------------------------------------------------------------------------------------------------------
// Fused gathered expert step (plain FFN): for every (group, 128-row tile of the tokens that keep it)
//   up projection -> bias, activation, selection bits -> H tile in shared memory -> down projection with the group's
//   columns of W2 -> the [rows, d] partial outputs are ADDED to a float32 accumulator at the rows of their tokens.
// This is the expert-major form of Listing 1 with its atomic merge (App. C): the hidden activations never leave the
// SM, nothing of the down projection is computed for pairs that were not kept, and the whole expert step costs time
// in proportion to the number of (token, group) pairs.  What bounds it on B200 is the merge: 4 d bytes of vector
// reductions per pair at about 5.5 TB/s for the whole chip, so it wins while few tokens keep a group.
// The caller pre-fills y32 with b2 and converts it to the output type afterwards (kernels below).
//
// 16 warps: scheduler, up-MMA issuer, down-MMA issuer, W2 producer (TMA), four gather warps, four warps for the first
// epilogue (up accumulator -> H tile) and four for the second (down accumulator -> staged, row-contiguous
// red.global.add.v4.f32).  TMEM: two 128-column up accumulators and two 128-column down accumulators, so gs <= 128.
constexpr int F_SCHED = 0, F_MMA_UP = 1, F_MMA_DN = 2, F_W2 = 3, F_GATHER0 = 4, F_EPI1_0 = 8, F_EPI2_0 = 12;
constexpr int F_NTHREADS = 512;
constexpr int F_CHUNK = 128;                 // columns of y per down accumulator
constexpr int F_STG_ROW = 272;               // staged accumulator row: 64 floats + 16 bytes of padding

struct FfnParams {
    GatherParams g;                  // scheduler and gather part (g.H unused)
    float *y32;                      // [T, d]
    int n_chunks, kb2;               // ceil(d / 128), ceil(gs / 64)
};

template <int ACT>
__global__ void __launch_bounds__(F_NTHREADS, 1)
moe_gather_ffn_kernel(const __grid_constant__ CUtensorMap tm_w1, const __grid_constant__ CUtensorMap tm_w2, const FfnParams fp)
{
    const GatherParams &p = fp.g;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *hs = smem + (size_t)p.stages * p.stage_bytes;                    // H tile: kb2 x (128 rows x 128 B), swizzled
    uint8_t *w2s = hs + (size_t)fp.kb2 * A_BYTES;                             // two slots of kb2 W2 tiles (128 rows x 128 B)
    uint8_t *stg = w2s + (size_t)2 * fp.kb2 * A_BYTES;                        // 128 staged accumulator rows
    uint32_t *fifo = reinterpret_cast<uint32_t *>(stg + 128 * F_STG_ROW);     // [FIFO_CAP] token indices
    __shared__ uint64_t bar_full[MAX_STAGES], bar_empty[MAX_STAGES], tile_full[TR], tile_empty[TR];
    __shared__ uint64_t up_full[2], up_empty[2], h_full, h_empty, w2_full[2], w2_empty[2], dn_full[2], dn_empty[2];
    __shared__ TileDesc tdesc[TR];
    __shared__ uint32_t tmem_base_holder;
    __shared__ uint32_t live[64];
    __shared__ int tok_s[BM];                                                 // tokens of the tile the second epilogue works on
    __shared__ volatile int e2_rows, e2_ok;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nkb = (p.d + BK - 1) / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1 + N_GATHER_WARPS * 32);
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        for (int t = 0; t < TR; ++t) {
            mbar_init(smem_u32(&tile_full[t]), 1);
            mbar_init(smem_u32(&tile_empty[t]), N_GATHER_WARPS + 3 + 4 + 1);  // gather, two MMA warps, W2 producer, epilogue 1, leader of epilogue 2
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&up_full[b]), 1);
            mbar_init(smem_u32(&up_empty[b]), 4);
            mbar_init(smem_u32(&w2_full[b]), 1);
            mbar_init(smem_u32(&w2_empty[b]), 1);
            mbar_init(smem_u32(&dn_full[b]), 1);
            mbar_init(smem_u32(&dn_empty[b]), 4);
        }
        mbar_init(smem_u32(&h_full), 4);
        mbar_init(smem_u32(&h_empty), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == F_MMA_UP) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_holder)), "r"(512u)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_holder;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const long long n_sel_now = p.n_sel ? (long long)__ldcg(p.n_sel) : 0;
    const bool run = p.n_sel == nullptr || (n_sel_now > p.n_sel_min && n_sel_now <= p.n_sel_max);

    if (!run) {
        // another path does the work
    } else if (warp == F_SCHED) {
        run_scheduler(p, fifo, tile_full, tile_empty, tdesc, live, lane);
    } else if (warp == F_MMA_UP) {
        const uint32_t idesc = instr_desc_bf16(BM, p.gs);
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
            const uint32_t ub = ti & 1u, use = ti >> 1;
            ok = mbar_wait_warp(smem_u32(&up_empty[ub]), (use & 1u) ^ 1u, p.status);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            ok = mma_tile(smem, bar_full, bar_empty, &up_full[ub], tmem_base + ub * 128u, idesc, nkb, p.stages, p.stage_bytes, it, p.status);
        }
    } else if (warp == F_MMA_DN) {
        // down projection of each tile: A = the H tile, B = the group's columns of W2, 128 output columns at a time
        const uint32_t idesc = instr_desc_bf16(BM, F_CHUNK);
        uint32_t cg = 0;
        bool ok = true;
        for (uint32_t ti = 0; ok; ++ti) {
            const uint32_t sl = ti % TR;
            ok = mbar_wait_warp(smem_u32(&tile_full[sl]), (ti / TR) & 1u, p.status);
            if (!ok) break;
            const int n_rows = tdesc[sl].n_rows;
            __syncwarp();
            if (n_rows < 0) break;
            if (elect_one()) mbar_arrive(smem_u32(&tile_empty[sl]));
            ok = mbar_wait_warp(smem_u32(&h_full), ti & 1u, p.status);
            for (int c = 0; c < fp.n_chunks && ok; ++c, ++cg) {
                const uint32_t slot = cg & 1u, use = cg >> 1;
                ok = mbar_wait_warp(smem_u32(&w2_full[slot]), use & 1u, p.status) &&
                     mbar_wait_warp(smem_u32(&dn_empty[slot]), (use & 1u) ^ 1u, p.status);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                if (elect_one()) {
                    for (int k = 0; k < p.gs / UMMA_K; ++k) {
                        const int j = k >> 2;
                        const uint64_t koff = (uint64_t)(((k & 3) * UMMA_K * 2) >> 4);
                        const uint64_t da = smem_desc_sw128(smem_u32(hs + (size_t)j * A_BYTES)) + koff;
                        const uint64_t db = smem_desc_sw128(smem_u32(w2s + (size_t)(slot * fp.kb2 + j) * A_BYTES)) + koff;
                        umma_bf16(tmem_base + 256u + slot * 128u, da, db, idesc, k > 0 ? 1u : 0u);
                    }
                    umma_commit(smem_u32(&w2_empty[slot]));
                    umma_commit(smem_u32(&dn_full[slot]));
                    if (c == fp.n_chunks - 1) umma_commit(smem_u32(&h_empty));      // the H tile may be rewritten
                }
                __syncwarp();
            }
        }
    } else if (warp == F_W2) {
        if (lane == 0) {
            uint32_t cg = 0;
            bool ok = true;
            for (uint32_t ti = 0; ok; ++ti) {
                const uint32_t sl = ti % TR;
                ok = mbar_wait(smem_u32(&tile_full[sl]), (ti / TR) & 1u, p.status);
                if (!ok) break;
                const int n_rows = tdesc[sl].n_rows, G = tdesc[sl].group;
                if (n_rows < 0) break;
                mbar_arrive(smem_u32(&tile_empty[sl]));
                for (int c = 0; c < fp.n_chunks && ok; ++c, ++cg) {
                    const uint32_t slot = cg & 1u, use = cg >> 1;
                    ok = mbar_wait(smem_u32(&w2_empty[slot]), (use & 1u) ^ 1u, p.status);
                    if (!ok) break;
                    const uint32_t full = smem_u32(&w2_full[slot]);
                    mbar_expect_tx(full, (uint32_t)(fp.kb2 * A_BYTES));
                    for (int j = 0; j < fp.kb2; ++j)
                        tma_load_2d(smem_u32(w2s + (size_t)(slot * fp.kb2 + j) * A_BYTES), &tm_w2, G * p.gs + j * BK, c * F_CHUNK, full);
                }
            }
        }
    } else if (warp >= F_GATHER0 && warp < F_EPI1_0) {
        // ---- gather warps: as in the up-projection kernel
        const int gw = warp - F_GATHER0, tid_g = gw * 32 + lane;
        const int chunk = tid_g & 7, rbase = tid_g >> 3;
        const uint32_t swz = (uint32_t)(((chunk ^ (rbase & 7)) << 4) + (rbase & 7) * 128 + (rbase >> 3) * 1024);
        uint32_t it = 0;
        bool ok = true;
        for (uint32_t ti = 0; ok; ++ti) {
            const uint32_t sl = ti % TR;
            ok = mbar_wait_warp(smem_u32(&tile_full[sl]), (ti / TR) & 1u, p.status);
            if (!ok) break;
            const int start = tdesc[sl].start, n_rows = tdesc[sl].n_rows, G = tdesc[sl].group;
            if (n_rows < 0) break;
            const __nv_bfloat16 *src[PASSES];
#pragma unroll
            for (int j = 0; j < PASSES; ++j) {
                const int r = rbase + ROWS_PER_PASS * j;
                src[j] = r < n_rows ? p.x + (size_t)fifo[(uint32_t)(start + r) % FIFO_CAP] * p.d + chunk * 8 : nullptr;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&tile_empty[sl]));
            for (int kb = 0; kb < nkb; ++kb, ++it) {
                const uint32_t s = it % (uint32_t)p.stages, round = it / (uint32_t)p.stages;
                ok = mbar_wait_warp(smem_u32(&bar_empty[s]), (round & 1u) ^ 1u, p.status);
                if (!ok) break;
                const uint32_t stage = smem_u32(smem + (size_t)s * p.stage_bytes), full = smem_u32(&bar_full[s]);
                if (gw == 0 && elect_one()) {
                    mbar_expect_tx(full, (uint32_t)(p.stage_bytes - A_BYTES));
                    tma_load_2d(stage + A_BYTES, &tm_w1, kb * BK, G * p.gs, full);
                }
                const bool in_k = kb * BK + chunk * 8 < p.d;
#pragma unroll
                for (int j = 0; j < PASSES; ++j) {
                    const bool live_row = in_k && src[j] != nullptr;
                    cp_async16(stage + swz + (uint32_t)(j * ROWS_PER_PASS * 128), live_row ? src[j] + kb * BK : p.x, live_row ? 16u : 0u);
                }
                cp_async_arrive(full);
            }
        }
        cp_async_wait_all();
    } else if (warp >= F_EPI1_0 && warp < F_EPI2_0) {
        // ---- epilogue 1: up accumulator -> bias, activation, selection bits -> bf16 H tile (swizzled K-major A operand)
        const int quad = warp & 3, row = quad * 32 + lane;
        const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
        const int n_units = p.gs >> 4;
        const bool halves = (p.s & 7) == 0;
        bool ok = true;
        for (uint32_t ti = 0; ok; ++ti) {
            const uint32_t sl = ti % TR;
            ok = mbar_wait_warp(smem_u32(&tile_full[sl]), (ti / TR) & 1u, p.status);
            if (!ok) break;
            const int start = tdesc[sl].start, n_rows = tdesc[sl].n_rows, G = tdesc[sl].group;
            if (n_rows < 0) break;
            const bool valid = row < n_rows;
            const uint32_t tok = valid ? fifo[(uint32_t)(start + row) % FIFO_CAP] : 0u;
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&tile_empty[sl]));
            const int e0 = G * p.g;
            const uint32_t bits = valid ? __ldg(p.mask + (size_t)tok * p.W + (e0 >> 5)) >> (e0 & 31) : 0u;     // rows past the end keep nothing
            const __nv_bfloat16 *brow = p.b1 ? p.b1 + (size_t)G * p.gs : nullptr;
            const uint32_t ub = ti & 1u, use = ti >> 1;
            ok = mbar_wait_warp(smem_u32(&up_full[ub]), use & 1u, p.status) &&
                 mbar_wait_warp(smem_u32(&h_empty), (ti & 1u) ^ 1u, p.status);          // the previous tile's down projection has read H
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t tbase = tmem_base + ub * 128u + lane_base;
            for (int u = 0; u < n_units; ++u) {
                const int c0 = u * 16;
                uint32_t ra[16];
                tmem_ld16_issue(tbase + (uint32_t)c0, ra);
                float bias[16];
                if (brow) {
                    float b8[8];
                    d2d_load8(brow + c0, b8);
#pragma unroll
                    for (int q = 0; q < 8; ++q) bias[q] = b8[q];
                    d2d_load8(brow + c0 + 8, b8);
#pragma unroll
                    for (int q = 0; q < 8; ++q) bias[8 + q] = b8[q];
                } else {
#pragma unroll
                    for (int q = 0; q < 16; ++q) bias[q] = 0.0f;
                }
                uint32_t keep;
                if (halves) {
                    const uint32_t e_lo = __umulhi((uint32_t)c0, p.inv_s), e_hi = __umulhi((uint32_t)(c0 + 8), p.inv_s);
                    keep = ((bits >> e_lo) & 1u ? 0x00ffu : 0u) | ((bits >> e_hi) & 1u ? 0xff00u : 0u);
                } else {
                    keep = 0u;
#pragma unroll
                    for (int j = 0; j < 16; ++j) keep |= ((bits >> __umulhi((uint32_t)(c0 + j), p.inv_s)) & 1u) << j;
                }
                tmem_ld_wait();
                uint32_t pk[8];
#pragma unroll
                for (int j = 0; j < 16; j += 2) {
                    const uint64_t z = add2(pack2(__uint_as_float(ra[j]), __uint_as_float(ra[j + 1])), pack2(bias[j], bias[j + 1]));
                    float v0, v1;
                    unpack2(fast_act2<ACT>(z), v0, v1);
                    const __nv_bfloat162 t2 = __floats2bfloat162_rn(v0, v1);
                    uint32_t wv = *reinterpret_cast<const uint32_t *>(&t2);
                    wv = (keep >> j) & 1u ? wv : (wv & 0xffff0000u);
                    wv = (keep >> (j + 1)) & 1u ? wv : (wv & 0x0000ffffu);
                    pk[j >> 1] = wv;
                }
                const int kb = c0 >> 6, ch = (c0 & 63) >> 3;
                uint8_t *rowp = hs + (size_t)kb * A_BYTES + (size_t)row * 128;
                *reinterpret_cast<uint4 *>(rowp + ((ch ^ (row & 7)) << 4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                *reinterpret_cast<uint4 *>(rowp + (((ch + 1) ^ (row & 7)) << 4)) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
            }
            // the accumulator is drained, the H tile is written: hand both on
            fence_async_smem();
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(smem_u32(&up_empty[ub]));
                mbar_arrive(smem_u32(&h_full));
            }
        }
    } else {
        // ---- epilogue 2: down accumulator -> staged rows -> row-contiguous vector reductions into y32 at the tokens' rows.
        // The four warps meet at named barriers, so every wait is done by one thread and its outcome shared.
        const int quad = warp & 3, row = quad * 32 + lane, wq = warp - F_EPI2_0;
        const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
        const bool leader = warp == F_EPI2_0 && lane == 0;
        uint32_t cg = 0;
        for (uint32_t ti = 0;; ++ti) {
            const uint32_t sl = ti % TR;
            if (leader) {
                const bool got = mbar_wait(smem_u32(&tile_full[sl]), (ti / TR) & 1u, p.status);
                e2_ok = got ? 1 : 0;
                e2_rows = got ? tdesc[sl].n_rows : -1;
            }
            asm volatile("bar.sync 2, 128;" ::: "memory");
            const int n_rows = e2_rows;
            if (!e2_ok || n_rows < 0) break;
            const int start = tdesc[sl].start;
            if (row < n_rows) tok_s[row] = (int)fifo[(uint32_t)(start + row) % FIFO_CAP];
            asm volatile("bar.sync 2, 128;" ::: "memory");
            if (leader) mbar_arrive(smem_u32(&tile_empty[sl]));
            bool ok = true;
            for (int c = 0; c < fp.n_chunks; ++c, ++cg) {
                const uint32_t slot = cg & 1u, use = cg >> 1;
                if (leader) e2_ok = mbar_wait(smem_u32(&dn_full[slot]), use & 1u, p.status) ? 1 : 0;
                asm volatile("bar.sync 2, 128;" ::: "memory");
                ok = e2_ok != 0;
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
                for (int hlf = 0; hlf < F_CHUNK / 64; ++hlf) {
                    uint32_t ra[4][16];
#pragma unroll
                    for (int u = 0; u < 4; ++u) tmem_ld16_issue(tmem_base + 256u + slot * 128u + lane_base + (uint32_t)(hlf * 64 + u * 16), ra[u]);
                    tmem_ld_wait();
                    if (row < n_rows) {
                        uint4 *o = reinterpret_cast<uint4 *>(stg + (size_t)row * F_STG_ROW);
#pragma unroll
                        for (int u = 0; u < 4; ++u)
#pragma unroll
                            for (int j = 0; j < 16; j += 4) o[u * 4 + (j >> 2)] = make_uint4(ra[u][j], ra[u][j + 1], ra[u][j + 2], ra[u][j + 3]);
                    }
                    asm volatile("bar.sync 2, 128;" ::: "memory");
                    const int col = c * F_CHUNK + hlf * 64 + (lane & 15) * 4;
                    for (int r = 2 * wq + (lane >> 4); r < n_rows; r += 8) {
                        const float4 v = *reinterpret_cast<const float4 *>(stg + (size_t)r * F_STG_ROW + (lane & 15) * 16);
                        if (col < p.d)
                            asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(fp.y32 + (size_t)tok_s[r] * p.d + col), "f"(v.x),
                                         "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
                    }
                    asm volatile("bar.sync 2, 128;" ::: "memory");
                }
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&dn_empty[slot]));
            }
            if (!ok) break;
        }
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == F_MMA_UP) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
}

// y32[t, :] = b2 before the fused kernel, y = bf16(y32) after it; both follow the fused kernel's dispatch rule
__global__ void __launch_bounds__(256)
y32_fill_kernel(float *__restrict__ y32, const __nv_bfloat16 *__restrict__ b2, long long total, int d, const int32_t *n_sel,
                long long n_sel_min, long long n_sel_max)
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (n_sel) {
        const long long n = (long long)__ldcg(n_sel);
        if (!(n > n_sel_min && n <= n_sel_max)) return;
    }
    // one float4 per thread and step, four steps in flight; the column of a float4 by 32-bit arithmetic
    const unsigned int q_total = (unsigned int)(total >> 2), q_row = (unsigned int)(d >> 2), stride = gridDim.x * 256u;
    for (unsigned int q0 = blockIdx.x * 256u + threadIdx.x; q0 < q_total; q0 += 4u * stride) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const unsigned int q = q0 + (unsigned int)u * stride;
            if (q >= q_total) break;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (b2) {
                const uint2 w = __ldg(reinterpret_cast<const uint2 *>(b2) + q % q_row);
                const __nv_bfloat162 lo = *reinterpret_cast<const __nv_bfloat162 *>(&w.x), hi = *reinterpret_cast<const __nv_bfloat162 *>(&w.y);
                v = make_float4(__low2float(lo), __high2float(lo), __low2float(hi), __high2float(hi));
            }
            __stcs(reinterpret_cast<float4 *>(y32) + q, v);
        }
    }
}

__global__ void __launch_bounds__(256)
y32_convert_kernel(const float *__restrict__ y32, __nv_bfloat16 *__restrict__ y, long long total, const int32_t *n_sel, long long n_sel_min,
                   long long n_sel_max)
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (n_sel) {
        const long long n = (long long)__ldcg(n_sel);
        if (!(n > n_sel_min && n <= n_sel_max)) return;
    }
    const unsigned int q_total = (unsigned int)(total >> 2), stride = gridDim.x * 256u;
    for (unsigned int q0 = blockIdx.x * 256u + threadIdx.x; q0 < q_total; q0 += 4u * stride) {
        float4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const unsigned int q = q0 + (unsigned int)u * stride;
            if (q < q_total) v[u] = __ldcs(reinterpret_cast<const float4 *>(y32) + q);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const unsigned int q = q0 + (unsigned int)u * stride;
            if (q >= q_total) break;
            const __nv_bfloat162 lo = __floats2bfloat162_rn(v[u].x, v[u].y), hi = __floats2bfloat162_rn(v[u].z, v[u].w);
            uint2 o;
            o.x = *reinterpret_cast<const uint32_t *>(&lo);
            o.y = *reinterpret_cast<const uint32_t *>(&hi);
            reinterpret_cast<uint2 *>(y)[q] = o;
        }
    }
}

bool ensure_attr(const void *kern, bool (&done)[64])
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
    if (!__atomic_load_n(&done[dev], __ATOMIC_ACQUIRE)) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 208 * 1024) != cudaSuccess) return false;
        __atomic_store_n(&done[dev], true, __ATOMIC_RELEASE);
    }
    return true;
}

template <int ACT, bool GATED>
d2d_status launch(const d2d_gather_args &a, cudaStream_t st)
{
    const int gs = a.g * a.s;
    const int b_rows = GATED ? 2 * gs : gs;
    GatherParams p = {};
    p.x = (const __nv_bfloat16 *)a.x; p.mask = a.mask; p.b1 = (const __nv_bfloat16 *)a.b1; p.H = (__nv_bfloat16 *)a.H;
    p.status = a.status; p.ctr = a.ctr; p.n_sel = a.n_sel; p.n_sel_min = a.n_sel_min; p.n_sel_max = a.n_sel_max;
    p.T = a.T; p.d = a.d; p.d_ff = a.d_ff; p.W = (a.n_experts + 31) / 32;
    p.g = a.g; p.s = a.s; p.gs = gs; p.n_groups = a.n_experts / a.g;
    p.inv_s = (uint32_t)((0x100000000ull + (unsigned long long)a.s - 1) / (unsigned long long)a.s);
    p.stage_bytes = A_BYTES + b_rows * 128;
    int stages = (192 * 1024) / p.stage_bytes;
    p.stages = stages > MAX_STAGES ? MAX_STAGES : stages;
    // about 48 MB of weight rows in flight: the rest of L2 holds the token rows and the outputs
    const long long group_bytes = (long long)b_rows * a.d * 2;
    long long window = (48ll << 20) / (group_bytes > 0 ? group_bytes : 1);
    p.window = (int)(window < 4 ? 4 : window > p.n_groups ? p.n_groups : window);
    if (p.window > p.n_groups) p.window = p.n_groups;
    p.visit_tiles = 8.0f;
    // tokens per draw: about eight draws per CTA (the CTAs then finish together), 256 .. 1024
    const long long want = (long long)a.T * p.n_groups / (8ll * d2d_tc_sm_count());
    p.sub = want >= 1024 ? 1024 : want >= 512 ? 512 : 256;
    const size_t smem = (size_t)p.stages * p.stage_bytes + FIFO_CAP * 4 + 1024;      // at most 192 + 8 + 1 KB
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
    if (!ensure_attr((const void *)kern, attr_set)) return D2D_ERR_CUDA;
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
    if (!d2d_moe_down_masked_supports(D)) return 0;           // the gathered kernel's H needs the down projection that reads only kept cells
    const int max_cols = D.gated ? 128 : 256;                 // one MMA holds gs (gated: 2 gs) accumulator columns
    auto fits = [&](int g) {
        const int gs = g * D.expert_size;
        return g >= 1 && g <= 32 && D.n_experts % g == 0 && 32 % g == 0 && gs % 16 == 0 && gs >= 16 && gs <= max_cols;
    };
    if (want > 0) return fits(want) ? want : 0;
    // default: the widest group one MMA can hold.  The kernel is bound by the rate at which token rows can be gathered
    // (about the same time per 128 x 64 tile of x whatever the width of the MMA that consumes it), so the more columns
    // a gathered row serves the better, although a wider group is kept by more tokens.
    for (int g = 32; g >= 1; g >>= 1)
        if (fits(g)) return g;
    return 0;
}

d2d_status d2d_moe_gather_up(const d2d_gather_args &a, cudaStream_t st)
{
    if (a.T <= 0) return D2D_OK;
    if (a.g < 1 || a.g > 32 || a.n_experts > 2048) return D2D_ERR_UNSUPPORTED;
    return a.w_gate ? launch_act<true>(a, st) : launch_act<false>(a, st);
}

bool d2d_moe_down_masked_supports(const d2d_layer_desc &D)
{
    return D.dtype == D2D_BF16 && D.d % 16 == 0 && D.d_ff % 8 == 0 && D.expert_size % 8 == 0 && D.d_ff < 65536 && d2d_gemm_tc_available();
}

d2d_status d2d_moe_down_masked(const d2d_layer_desc &D, const void *H, const uint32_t *mask, const void *w2, const void *b2, void *y, int T,
                               int32_t *status, cudaStream_t st, const int32_t *n_sel, long long n_sel_min, long long n_sel_max)
{
    if (T <= 0) return D2D_OK;
    if (!d2d_moe_down_masked_supports(D)) return D2D_ERR_UNSUPPORTED;
    const int sms = d2d_tc_sm_count();
    // column tile that wastes the fewest SM rounds (wider preferred on ties: fewer passes over H)
    int bn = 256;
    double best = -1.0;
    for (int cand : {256, 192, 128}) {
        const long tiles = (long)d2d_cdiv(D.d, cand) * d2d_cdiv(T, BM);
        const long rounds = (tiles + sms - 1) / sms;
        const double eff = (double)D.d / ((double)d2d_cdiv(D.d, cand) * cand) * (double)tiles / (double)(rounds * sms);
        if (eff > best + 1e-9) { best = eff; bn = cand; }
    }
    DownParams p = {};
    p.H = (const __nv_bfloat16 *)H; p.mask = mask; p.b2 = (const __nv_bfloat16 *)b2; p.y = (__nv_bfloat16 *)y; p.status = status;
    p.T = T; p.d = D.d; p.d_ff = D.d_ff; p.W = (D.n_experts + 31) / 32; p.s = D.expert_size;
    p.inv_s = (uint32_t)((0x100000000ull + (unsigned long long)D.expert_size - 1) / (unsigned long long)D.expert_size);
    p.bn = bn;
    p.n_sel = n_sel; p.n_sel_min = n_sel_min; p.n_sel_max = n_sel_max;
    p.stage_bytes = A_BYTES + bn * 128;
    const int stages = (192 * 1024) / p.stage_bytes;
    p.stages = stages > MAX_STAGES ? MAX_STAGES : stages;
    // W2 of Llama-sized layers does not stay in L2 beside H: walk the tiles in bands of about 32 MB of H rows
    p.band = 0;
    if (2.0 * D.d * D.d_ff >= 48e6) {
        const int band = (int)(32e6 / (2.0 * BM * D.d_ff) + 0.5);
        p.band = band < 16 ? 16 : band;
    }
    const size_t smem = (size_t)p.stages * p.stage_bytes + 1024;
    CUtensorMap tw2;
    if (!d2d_tc_make_map(&tw2, w2, D.d, D.d_ff, bn)) return D2D_ERR_CUDA;
    static bool attr_set[64] = {};
    if (!ensure_attr((const void *)moe_down_masked_kernel, attr_set)) return D2D_ERR_CUDA;
    const int tiles = d2d_cdiv(D.d, bn) * d2d_cdiv(T, BM);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(tiles < sms ? tiles : sms, 1, 1);
    cfg.blockDim = dim3(NTHREADS, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = d2d_tc_pdl_enabled() ? 1 : 0;
    const cudaError_t err = cudaLaunchKernelEx(&cfg, moe_down_masked_kernel, tw2, p);
    D2D_LAUNCHED(1);
    return err == cudaSuccess && cudaGetLastError() == cudaSuccess ? D2D_OK : D2D_ERR_CUDA;
}

// Zero for the cells of H that the gathered up projection leaves alone: (token, group) pairs without a kept expert.
// With them H is fully defined and the plain TMA-fed dense down projection can follow (10-20 % faster than the one
// that applies the selection while it stages H); the price is (1 - u) T d_ff 2 bytes of stores at memory bandwidth,
// which pays for wide layers (the down projection's time grows with d, the fill's does not).
// One thread per 16-byte chunk: consecutive lanes write consecutive chunks of a token's row.
__global__ void __launch_bounds__(256)
h_zero_unkept_kernel(__nv_bfloat16 *__restrict__ H, const uint32_t *__restrict__ mask, int T, int W, int d_ff, int g, uint32_t inv_gs,
                     const int32_t *n_sel, long long n_sel_min, long long n_sel_max)
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (n_sel) {
        const long long n = (long long)__ldcg(n_sel);
        if (!(n > n_sel_min && n <= n_sel_max)) return;
    }
    const int chunks = d_ff >> 3;
    const uint32_t gm = g >= 32 ? 0xffffffffu : (1u << g) - 1u;
    const long long total = (long long)T * chunks;
    for (long long i = (long long)blockIdx.x * 256 + threadIdx.x; i < total; i += (long long)gridDim.x * 256) {
        const int t = (int)(i / chunks), c = (int)(i - (long long)t * chunks);
        const int e0 = (int)__umulhi((uint32_t)(c * 8), inv_gs) * g;              // first expert of the chunk's group
        const uint32_t bits = (__ldg(mask + (size_t)t * W + (e0 >> 5)) >> (e0 & 31)) & gm;
        if (bits == 0u) *reinterpret_cast<uint4 *>(H + (size_t)t * d_ff + (size_t)c * 8) = make_uint4(0u, 0u, 0u, 0u);
    }
}

d2d_status d2d_moe_zero_unkept(void *H, const uint32_t *mask, int T, int d_ff, int n_experts, int s, int g, const int32_t *n_sel,
                               long long n_sel_min, long long n_sel_max, cudaStream_t st)
{
    if (T <= 0) return D2D_OK;
    const int gs = g * s;
    if (g < 1 || g > 32 || 32 % g || n_experts % g || gs % 8 || d_ff % 8) return D2D_ERR_UNSUPPORTED;
    const uint32_t inv_gs = (uint32_t)((0x100000000ull + (unsigned long long)gs - 1) / (unsigned long long)gs);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = d2d_tc_pdl_enabled() ? 1 : 0;
    const long long total = (long long)T * (d_ff / 8);
    const long long blocks = (total + 255) / 256;
    const int cap = 16 * d2d_tc_sm_count();
    cfg.gridDim = dim3((unsigned)(blocks < cap ? blocks : cap), 1, 1);
    cfg.blockDim = dim3(256, 1, 1);
    const cudaError_t err = cudaLaunchKernelEx(&cfg, h_zero_unkept_kernel, (__nv_bfloat16 *)H, mask, T, (n_experts + 31) / 32, d_ff, g, inv_gs,
                                               n_sel, n_sel_min, n_sel_max);
    D2D_LAUNCHED(1);
    return err == cudaSuccess && cudaGetLastError() == cudaSuccess ? D2D_OK : D2D_ERR_CUDA;
}

int d2d_gather_ffn_group_for(const d2d_layer_desc &D)
{
    // the float32 accumulator [T, d] takes the place of H [T, d_ff] bf16 in the caller's workspace
    if (D.gated || !d2d_moe_down_masked_supports(D) || D.d % 8 || D.d < 128 || D.d > 128 * 32 || D.d_ff < 2 * D.d) return 0;
    for (int g = 32; g >= 1; g >>= 1) {
        const int gs = g * D.expert_size;
        if (D.n_experts % g == 0 && 32 % g == 0 && gs % 16 == 0 && gs >= 16 && gs <= 128) return g;
    }
    return 0;
}

template <int ACT>
static d2d_status launch_ffn(const d2d_gather_args &a, float *y32, void *y, const void *w2, const void *b2, cudaStream_t st)
{
    const int gs = a.g * a.s;
    FfnParams fp = {};
    GatherParams &p = fp.g;
    p.x = (const __nv_bfloat16 *)a.x; p.mask = a.mask; p.b1 = (const __nv_bfloat16 *)a.b1; p.H = nullptr;
    p.status = a.status; p.ctr = a.ctr; p.n_sel = a.n_sel; p.n_sel_min = a.n_sel_min; p.n_sel_max = a.n_sel_max;
    p.T = a.T; p.d = a.d; p.d_ff = a.d_ff; p.W = (a.n_experts + 31) / 32;
    p.g = a.g; p.s = a.s; p.gs = gs; p.n_groups = a.n_experts / a.g;
    p.inv_s = (uint32_t)((0x100000000ull + (unsigned long long)a.s - 1) / (unsigned long long)a.s);
    p.stage_bytes = A_BYTES + gs * 128;
    fp.y32 = y32;
    fp.n_chunks = d2d_cdiv(a.d, F_CHUNK);
    fp.kb2 = d2d_cdiv(gs, BK);
    const size_t fixed = (size_t)3 * fp.kb2 * A_BYTES + 128 * F_STG_ROW + FIFO_CAP * 4 + 1024;
    int stages = (int)((216 * 1024 - fixed) / p.stage_bytes);
    p.stages = stages > MAX_STAGES ? MAX_STAGES : stages;
    if (p.stages < 2) return D2D_ERR_UNSUPPORTED;
    const size_t smem = (size_t)p.stages * p.stage_bytes + fixed;
    p.window = p.n_groups;                                    // plain layers: all weights of these shapes fit in L2
    const long long group_bytes = (long long)gs * a.d * 4;    // W1 rows and W2 columns of a group
    long long window = (48ll << 20) / (group_bytes > 0 ? group_bytes : 1);
    p.window = (int)(window < 4 ? 4 : window > p.n_groups ? p.n_groups : window);
    if (p.window > p.n_groups) p.window = p.n_groups;
    p.visit_tiles = 8.0f;
    const long long want = (long long)a.T * p.n_groups / (8ll * d2d_tc_sm_count());
    p.sub = want >= 1024 ? 1024 : want >= 512 ? 512 : 256;
    CUtensorMap tw1, tw2;
    if (!d2d_tc_make_map(&tw1, a.w1, a.d_ff, a.d, gs) || !d2d_tc_make_map(&tw2, w2, a.d, a.d_ff, 128)) return D2D_ERR_CUDA;
    auto kern = moe_gather_ffn_kernel<ACT>;
    static bool attr_set[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return D2D_ERR_CUDA;
    if (!__atomic_load_n(&attr_set[dev], __ATOMIC_ACQUIRE)) {
        if (cudaFuncSetAttribute((const void *)kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 217 * 1024) != cudaSuccess) return D2D_ERR_CUDA;
        __atomic_store_n(&attr_set[dev], true, __ATOMIC_RELEASE);
    }
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = d2d_tc_pdl_enabled() ? 1 : 0;
    const long long total = (long long)a.T * a.d;
    const int blocks = (int)((total / 4 + 255) / 256);
    const int sms = d2d_tc_sm_count();
    if (total / 4 >= (1ll << 31)) return D2D_ERR_UNSUPPORTED;
    cfg.gridDim = dim3(blocks < 8 * sms ? blocks : 8 * sms, 1, 1);
    cfg.blockDim = dim3(256, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cudaError_t err = cudaLaunchKernelEx(&cfg, y32_fill_kernel, y32, (const __nv_bfloat16 *)b2, total, a.d, a.n_sel, a.n_sel_min, a.n_sel_max);
    if (err == cudaSuccess) {
        cudaLaunchConfig_t kc = cfg;
        kc.gridDim = dim3(sms, 1, 1);
        kc.blockDim = dim3(F_NTHREADS, 1, 1);
        kc.dynamicSmemBytes = smem;
        err = cudaLaunchKernelEx(&kc, kern, tw1, tw2, fp);
    }
    if (err == cudaSuccess)
        err = cudaLaunchKernelEx(&cfg, y32_convert_kernel, (const float *)y32, (__nv_bfloat16 *)y, total, a.n_sel, a.n_sel_min, a.n_sel_max);
    D2D_LAUNCHED(3);
    return err == cudaSuccess && cudaGetLastError() == cudaSuccess ? D2D_OK : D2D_ERR_CUDA;
}

d2d_status d2d_moe_gather_ffn(const d2d_gather_args &a, float *y32, void *y, const void *w2, const void *b2, cudaStream_t st)
{
    if (a.T <= 0) return D2D_OK;
    if (a.w_gate || a.g < 1 || a.g > 32 || a.g * a.s > 128 || a.n_experts > 2048) return D2D_ERR_UNSUPPORTED;
    switch (a.act) {
    case D2D_ACT_RELU: return launch_ffn<D2D_ACT_RELU>(a, y32, y, w2, b2, st);
    case D2D_ACT_GELU_ERF: return launch_ffn<D2D_ACT_GELU_ERF>(a, y32, y, w2, b2, st);
    case D2D_ACT_GELU_TANH: return launch_ffn<D2D_ACT_GELU_TANH>(a, y32, y, w2, b2, st);
    case D2D_ACT_SILU: return launch_ffn<D2D_ACT_SILU>(a, y32, y, w2, b2, st);
    }
    return D2D_ERR_INVALID_ARG;
}
