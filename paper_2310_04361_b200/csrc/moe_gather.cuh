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
    void *H;                 // [T, d_ff] bf16; only the cells of kept (token, group) pairs are written (inside such a cell,
                             // the neurons of experts the token did not keep are zero); feed it to d2d_moe_down_masked
    int T, d, d_ff, n_experts;
    int s;                   // expert size
    int g;                   // experts per group (from d2d_gather_group_for)
    int act;                 // d2d_act
    int32_t *status;         // device status word (D2D_ERR_TIMEOUT)
    int *ctr;                // n_experts / g + 1 device ints, zero before the first launch; the kernel leaves them at zero
    // Density-adaptive dispatch without a host synchronisation: when n_sel is given, the kernel reads the number of
    // selected pairs of this batch from it and works only if n_sel_min < n_sel <= n_sel_max, returning at once
    // otherwise (the caller launches the other paths with the complementary rules; -1 and LLONG_MAX = always run).
    // The kernel also sizes its work distribution from that density.  NULL = always run, distribution sized for
    // dense selections.
    const int32_t *n_sel;
    long long n_sel_min, n_sel_max;
};

// Experts per group for this layer shape: `want` if it is usable (0 = pick the default), 0 if the gathered path
// cannot serve the shape (fp32 layers, expert sizes that are not multiples of 8, groups wider than one MMA).
int d2d_gather_group_for(const d2d_layer_desc &D, int want);

d2d_status d2d_moe_gather_up(const d2d_gather_args &a, cudaStream_t st);

// Down projection that applies the selection while it stages H: y = (G * H) W2^T + b2, reading only the cells of H
// whose (token, expert) pair is kept.  Follows d2d_moe_gather_up (which writes only those cells) and is equally valid
// after the masked dense up projection.  w2: [d, d_ff] bf16 as given; requires d % 16 == 0 and s % 8 == 0.
bool d2d_moe_down_masked_supports(const d2d_layer_desc &D);
// n_sel / n_sel_min / n_sel_max: as in d2d_gather_args (NULL = always run).
d2d_status d2d_moe_down_masked(const d2d_layer_desc &D, const void *H, const uint32_t *mask, const void *w2, const void *b2, void *y, int T,
                               int32_t *status, cudaStream_t st, const int32_t *n_sel = nullptr, long long n_sel_min = -1,
                               long long n_sel_max = 0);

// Fused gathered expert step of plain (not gated) layers: up projection, activation, down projection and the
// scatter-add of the partial outputs per (group, tile of the tokens that keep it), see moe_gather.cu.  a.H is unused,
// a.g must come from d2d_gather_ffn_group_for (groups of at most 128 neurons).  y32: [T, d] float32 scratch (caller's),
// filled with b2, accumulated into with vector reductions and converted to y [T, d] bf16: three launches, all
// following the dispatch rule in `a`.
int d2d_gather_ffn_group_for(const d2d_layer_desc &D);
d2d_status d2d_moe_gather_ffn(const d2d_gather_args &a, float *y32, void *y, const void *w2, const void *b2, cudaStream_t st);

// Writes zero to the cells of H [T, d_ff] bf16 of (token, group) pairs without a kept expert: what the gathered up
// projection (groups of g experts) does not write.  Afterwards H is fully defined.  Follows the dispatch rule.
d2d_status d2d_moe_zero_unkept(void *H, const uint32_t *mask, int T, int d_ff, int n_experts, int s, int g, const int32_t *n_sel,
                               long long n_sel_min, long long n_sel_max, cudaStream_t st);
