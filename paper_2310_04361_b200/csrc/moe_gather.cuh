// Interface of the gathered, grouped expert up projection (see moe_gather.cu).
#pragma once

#include "d2d_common.cuh"
#include "gemm_tc.cuh"

struct d2d_gather_args {
    const void *x;           // [T, d] bf16 token rows
    const void *w1;          // [d_ff, d] bf16 (an expert = s contiguous rows)
    const void *w_gate;      // [d_ff, d] bf16 or NULL
    const void *b1;          // [d_ff] bf16 or NULL
    const uint32_t *mask;    // [T, ceil(E/32)] selection mask
    void *H;                 // [T, d_ff] bf16, every element is written (kept experts: activations, others: zeros)
    int T, d, d_ff, n_experts;
    int s;                   // expert size
    int g;                   // experts per group (from d2d_gather_group_for)
    int act;                 // d2d_act
    int32_t *status;         // device status word (D2D_ERR_TIMEOUT)
    int *ctr;                // n_experts / g + 1 device ints, zero before the first launch; the kernel leaves them at zero
    // Density-adaptive dispatch without a host synchronisation: when n_sel is given, the kernel reads the number of
    // selected pairs of this batch from it and returns at once if it exceeds n_sel_max (the caller launches the
    // masked dense up projection with the complementary rule).  NULL = always run.
    const int32_t *n_sel;
    long long n_sel_max;
};

// Experts per group for this layer shape: `want` if it is usable (0 = pick the default), 0 if the gathered path
// cannot serve the shape (fp32 layers, expert sizes that are not multiples of 8, groups wider than one MMA).
int d2d_gather_group_for(const d2d_layer_desc &D, int want);

d2d_status d2d_moe_gather_up(const d2d_gather_args &a, cudaStream_t st);
