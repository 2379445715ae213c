// Interface of the tcgen05 / TMA GEMM used for the dense contractions of the layer
// (router layers, expert up projection with fused bias + activation + mask, down projection).
#pragma once

#include <cuda.h>

#include "d2d_common.cuh"

enum d2d_gemm_epilogue {
    D2D_EPI_RELU_BF16 = 0,   // out bf16 = relu(acc + bias)                 router layer 1
    D2D_EPI_ABS_F32 = 1,     // out f32  = |acc + bias|                     router layer 2
    D2D_EPI_UP_MASKED = 2,   // out bf16 = G[row, col/s] ? A(acc + bias) : 0    expert up projection
    D2D_EPI_BIAS_BF16 = 3,   // out bf16 = acc + bias                       down projection
    D2D_EPI_PARTIAL_F32 = 4, // out f32 += acc (vector reductions)          one K slice of a split-K GEMM (internal)
};

struct d2d_gemm_args {
    const void *a;           // [M, K] bf16 row-major (activations)
    const void *b;           // [N, K] bf16 row-major (weights, nn.Linear layout)
    const void *b_gate;      // [N, K] second weight matrix for the gated up projection, else NULL
    // optional copy of b and b_gate interleaved in blocks of b_cat_block rows: [b rows of block 0 | gate rows of block 0 |
    // b rows of block 1 | ...], the last block zero padded; lets the gated kernel fetch both tiles with one load
    const void *b_cat;
    int b_cat_block;
    const void *bias;        // [N] bf16 or NULL
    void *out;               // [M, N] bf16 or f32, row-major, leading dimension N
    int M, N, K;
    int epilogue;            // d2d_gemm_epilogue
    int act;                 // d2d_act, used by D2D_EPI_UP_MASKED
    const uint32_t *mask;    // [M, mask_words] packed selection mask (UP_MASKED), NULL = keep everything
    int mask_words;
    int expert_size;         // s: column c belongs to expert c / s
    int32_t *status;         // device status word, receives D2D_ERR_TIMEOUT if a bounded wait runs out
    // Split-K (D2D_EPI_BIAS_BF16 only): with k_splits > 1 the K range is cut into slices that run as separate work
    // items, partial sums meet in `partial` (float32 [M, N], cleared by the call), a small kernel adds the bias and
    // converts.  For problems with so few output tiles that most SMs would idle (decode batches).
    int k_splits;
    float *partial;
    // Dynamic tile scheduling: a device counter that is ZERO when the kernel starts; CTAs draw work items from it
    // instead of walking a fixed round-robin list, and the last draw of a launch resets it to zero (a launch that ends
    // in D2D_ERR_TIMEOUT may leave it non-zero).  NULL = static schedule.
    int *tile_counter;
    // 1: A, B and the bias do NOT depend on the previous kernel of the stream, only the epilogue inputs (the selection
    // mask) do.  With programmatic dependent launch the main loops then start while that kernel still runs and only the
    // epilogue waits for it.  Never set this when A may be written by the preceding kernel.
    int pdl_late_wait;
    // Batched problems with one shape (the down projections of several layers that ran as one merged up projection):
    // with batch > 1, A is [M, batch*K] and problem p reads its columns [p*K, (p+1)*K); B is [batch*N, K] and bias is
    // [batch*N], problem p owns rows / entries [p*N, (p+1)*N); out is [batch, M, N] (problem p at out + p*M*N).
    // Requires K % 64 == 0.  0 and 1 both mean a single problem.
    int batch;
    // Density-adaptive dispatch (D2D_EPI_UP_MASKED): when n_sel is given the kernel reads the number of selected
    // (token, expert) pairs from it once the previous kernel of the stream has completed and returns without doing
    // anything if it is at most n_sel_max (the gathered kernel, launched with the complementary rule, does the
    // work).  Cannot be combined with pdl_late_wait.
    const int32_t *n_sel;
    long long n_sel_max;
    // Test aid for the failure-handling test (host-made fault, nothing traps or spins without bound): CTA 0 leaves out
    // the load of the A tile of its first k-block, so the barrier of that stage never completes; the bounded waits of
    // the MMA warp, the epilogue and the producer run out, D2D_ERR_TIMEOUT is recorded, every role reaches the final
    // barrier, TMEM is freed and the kernel returns.  Only honoured by the statically scheduled launch.
    int test_skip_load;
};

// Number of K slices d2d_gemm_tc would use for a [M,N,K] down projection (1 = no split) and the float32 scratch it needs.
int d2d_gemm_tc_splits(int M, int N, int K, int batch = 1);

// Enqueues C = epilogue(A B^T).  Requires K % 8 == 0 and 16-byte aligned base pointers.
d2d_status d2d_gemm_tc(const d2d_gemm_args &g, cudaStream_t st);

// False when the driver entry point for tensor-map encoding is unavailable.
bool d2d_gemm_tc_available();
