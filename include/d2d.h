/*
 * d2d.h - C ABI of the B200 (sm_100a) dynamic-k MoE layer library.
 *
 * The library runs the inference hot path of one D2DMoE layer
 * (arXiv 2310.04361): a dense Transformer FFN (plain or gated), or a MoE-fied
 * attention projection, whose neurons were cut offline into E equal experts
 * (Sec. 3.2) and that runs, per token, only the experts a small router keeps
 * (Sec. 3.3, 3.4).  The four steps are
 *
 *   router_fwd     R[t,i] = | W_r2 relu(W_r1 x_t + b_r1) + b_r2 |_i      Sec. 3.3
 *   select_dynk    G[t,i] = ( R[t,i] >= tau * max_i R[t,i] )             Eq. 4
 *                  + per-token k, per-expert counts, offsets, token lists  Listing 1
 *   moe_ffn_fwd    y_t = b2 + sum_{i: G[t,i]} W2[:, blk i] A(W1[blk i,:] x_t + b1[blk i])
 *                                                                         Sec. 3.2, App. G
 *
 * General rules
 *   - Every pointer named "device" is a CUDA device pointer on the current
 *     device; "host" pointers are ordinary host memory.  All matrices are
 *     row-major.  Weight matrices use the nn.Linear layout [out, in].
 *   - The caller owns every buffer it passes, including the workspace.  The
 *     library allocates device memory only inside d2d_layer_create (packed
 *     copies of the weights) and frees it in d2d_layer_destroy.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *     stream).  Calls enqueue work and return; none of them synchronises,
 *     except d2d_layer_create (once, after packing).
 *   - The return value reports argument and launch errors only.  Conditions
 *     that depend on the data (a non-finite router score, more selected pairs
 *     than `perm_capacity`) are written to the device status word
 *     `d2d_routing.status`, which the caller reads after synchronising.
 *   - T = 0 is a valid no-op.  There is no CPU fallback: without a CUDA device
 *     every compute call returns D2D_ERR_CUDA.
 *   - A handle is not thread-safe; distinct handles may be used concurrently.
 *
 * Environment variables (tuning aids, read once per process; results never
 * depend on them)
 *   D2D_DECODE_MAX_TOKENS=n  0..8: bf16 batches of up to n tokens take the decode
 *                            kernels (each kept expert's weights read once by CUDA
 *                            cores), larger ones the tensor-core path.  Default: 4
 *                            tokens, 2 for layers with more than 256 KB of weights
 *                            per expert.
 *   D2D_HOST_CHUNKS=n        1..4: number of pipelined chunks d2d_layer_fwd_host
 *                            cuts a batch into, of equal size (default: see there).
 *   D2D_GEMM_BAND=n          row tiles per band of the tile walk of the dense
 *                            kernels when the weight operand exceeds L2 (default:
 *                            about 32 MB of activation rows), 0 = row-major walk.
 *   D2D_GEMM_PDL=0           launch every kernel fully serialised (no programmatic
 *                            dependent launch).
 */
#ifndef D2D_H_
#define D2D_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define D2D_API __attribute__((visibility("default")))
#else
#define D2D_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    D2D_OK = 0,
    D2D_ERR_INVALID_ARG = 1, /* null pointer, bad size, tau outside [0,1], misaligned buffer */
    D2D_ERR_UNSUPPORTED = 2, /* a shape or option the kernels do not cover                  */
    D2D_ERR_WORKSPACE = 3,   /* workspace smaller than d2d_workspace_bytes reports          */
    D2D_ERR_CUDA = 4,        /* a CUDA runtime call or a launch failed                      */
    D2D_ERR_NONFINITE = 5,   /* device status: a router score was NaN or infinite           */
    D2D_ERR_TIMEOUT = 6,     /* device status: a bounded wait inside a kernel ran out       */
    D2D_ERR_CAPACITY = 7     /* device status: n_sel exceeded perm_capacity                 */
} d2d_status;

typedef enum { D2D_F32 = 0, D2D_BF16 = 1 } d2d_dtype;

/* Activation A of the hidden neurons.  The paper evaluates ReLU and GELU models
 * (Sec. 4, Sec. 5.4) and SiLU-gated FFNs (App. G); it does not say which GELU
 * form, so both are offered. */
typedef enum { D2D_ACT_RELU = 0, D2D_ACT_GELU_ERF = 1, D2D_ACT_GELU_TANH = 2, D2D_ACT_SILU = 3 } d2d_act;

/* Shape of one layer.  Expert e owns neurons [e*expert_size, (e+1)*expert_size)
 * (Sec. 3.2); n_experts * expert_size must equal d_ff.  d and d_h must be
 * multiples of 8 so that every matrix row starts on a 16-byte boundary. */
typedef struct {
    int32_t d;           /* model width (input and output of the layer)           */
    int32_t d_ff;        /* hidden width of the original FFN                       */
    int32_t n_experts;   /* E                                                      */
    int32_t expert_size; /* s = d_ff / E                                           */
    int32_t d_h;         /* router hidden width (Sec. 3.3; 128 in the paper)       */
    d2d_dtype dtype;     /* type of x, y and of every weight and bias              */
    d2d_act act;
    int32_t gated;       /* 0: y = W2 A(W1 x + b1) + b2                            */
                         /* 1: y = W2 (A(W_gate x) * (W1 x + b1)) + b2  (App. G)   */
} d2d_layer_desc;

/* Device pointers to the layer's parameters, element type desc.dtype, read
 * only during d2d_layer_create (the library keeps packed copies, so the
 * caller may free these afterwards).  Any bias pointer may be NULL (= zeros). */
typedef struct {
    const void *w_r1;   /* [d_h, d]      router layer 1                              */
    const void *b_r1;   /* [d_h]                                                     */
    const void *w_r2;   /* [E, d_h]      router layer 2 (absolute value on output)   */
    const void *b_r2;   /* [E]                                                       */
    const void *w1;     /* [d_ff, d]     first FFN matrix ("up" when gated)          */
    const void *b1;     /* [d_ff]                                                    */
    const void *w_gate; /* [d_ff, d]     gate matrix, required iff desc.gated        */
    const void *w2;     /* [d, d_ff]     second FFN matrix                           */
    const void *b2;     /* [d]           shared by all experts, added once per token */
} d2d_weights;

/* Routing of one batch: the outputs of d2d_select_dynk and the input of
 * d2d_moe_ffn_fwd.  All pointers are device pointers owned by the caller.
 * mask, k, counts, offsets, perm, n_sel and status are required; the
 * token-major dual (tok_off, tok_exp) is optional (both NULL or both set).
 * d2d_layer_fwd alone also accepts a routing whose per-expert lists are absent
 * as a set (counts, offsets, perm, n_sel, tok_off, tok_exp all NULL); see there. */
typedef struct {
    uint32_t *mask;      /* [T, ceil(E/32)]  expert i of token t = bit i%32 of word i/32       */
    int32_t *k;          /* [T]              experts kept by token t                           */
    int32_t *counts;     /* [E]              tokens that keep expert e                         */
    int32_t *offsets;    /* [E+1]            exclusive prefix sum of counts                    */
    int32_t *perm;       /* [perm_capacity]  perm[offsets[e]+j] = j-th smallest t keeping e    */
    int32_t *tok_off;    /* [T+1]            exclusive prefix sum of k            (optional)   */
    int32_t *tok_exp;    /* [perm_capacity]  experts of token t, ascending        (optional)   */
    int32_t *n_sel;      /* [1]              total kept (token, expert) pairs = offsets[E]     */
    int32_t *status;     /* [1]              device status word: 0 or a d2d_status             */
    int64_t perm_capacity; /* entries available in perm / tok_exp; T*E always suffices         */
} d2d_routing;

typedef struct d2d_layer d2d_layer;

/* Human-readable name of a status code (host, static storage). */
D2D_API const char *d2d_status_str(d2d_status s);

/* Number of kernels this library has launched in this process so far (host
 * counter, all handles and streams); a benchmark takes the difference across
 * its timed region. */
D2D_API uint64_t d2d_launch_count(void);

/* Builds a layer handle: validates `desc`, copies and repacks the weights on
 * the device (W2 is stored transposed so that an expert's slice is
 * expert_size contiguous rows of d elements) and synchronises `stream` once.
 * `desc` and `w` are host structs; the pointers inside `w` are device
 * pointers.  On failure *out is NULL. */
D2D_API d2d_status d2d_layer_create(const d2d_layer_desc *desc, const d2d_weights *w, void *stream, d2d_layer **out);

/* The same layer with 8-bit expert weights (App. C runs the expert kernels on
 * narrower number formats).  Every expert's slice of W1, W_gate and W2 is
 * rounded to 8-bit floating point codes (e4m3: 1 sign, 4 exponent, 3 mantissa
 * bits, bias 7, largest value 448; round to nearest, ties to even, saturating)
 * with ONE power-of-two scale 2^k per expert and matrix, k the smallest integer
 * for which the slice's largest magnitude fits (0 for an all-zero slice).  The
 * layer then computes with the rounded weights value(code) * 2^k on every path
 * (they are exactly bf16 values, kept in the packed bf16 copies); the decode
 * kernels read the codes, half the bytes per kept expert.  Router weights and
 * biases are not touched.  bf16 layers with d and expert_size * d multiples of
 * 16 only (D2D_ERR_UNSUPPORTED otherwise).  Costs d_ff * d bytes per matrix on
 * top of d2d_layer_create. */
D2D_API d2d_status d2d_layer_create_fp8(const d2d_layer_desc *desc, const d2d_weights *w, void *stream, d2d_layer **out);
/* Copies the codes (device uint8 [d_ff, d]; an expert = expert_size contiguous
 * rows; which = 2: of W2 transposed) and/or the exponents k (device int32 [E])
 * of which = 0: W1, 1: W_gate, 2: W2.  Either output may be NULL.
 * D2D_ERR_UNSUPPORTED for a layer without 8-bit weights (or without W_gate). */
D2D_API d2d_status d2d_layer_get_fp8(const d2d_layer *layer, int32_t which, uint8_t *codes, int32_t *exps, void *stream);

/* Frees the handle and its device copies.  NULL is a no-op. */
D2D_API d2d_status d2d_layer_destroy(d2d_layer *layer);

/* How the expert step of bf16 batches above the decode sizes computes the up
 * projection H = G * A(x W1^T + b1) (Sec. 3.4).  Both forms give the same H;
 * the choice changes speed only.
 *   D2D_PATH_DENSE   one contraction over all d_ff neurons with the selection
 *                    applied as a mask: time independent of the selection.
 *   D2D_PATH_GATHER  tokens are bucketed by groups of `group` adjacent experts
 *                    and each group runs a contraction over the tokens that keep
 *                    one of its experts (the grouped form of Listing 1): time
 *                    proportional to the number of kept (token, group) pairs.
 *   D2D_PATH_FUSED   (plain layers, groups of at most 128 neurons) one kernel per
 *                    (group, tile of the tokens that keep it): up projection,
 *                    activation, down projection with the group's columns of W2,
 *                    and the partial outputs added to a float32 accumulator [T, d]
 *                    with vector reductions (the atomic merge of App. C); the
 *                    accumulator lives where H would in the workspace, is filled
 *                    with b2 before and converted to y after.  H never exists and
 *                    the whole step is proportional to the kept pairs; the merge
 *                    bounds it, so it wins only at low densities.  The order of
 *                    the float32 additions is not fixed: y may differ from run to
 *                    run in the last bits.
 *   D2D_PATH_AUTO    (default) decided per call on the device from the number of
 *                    selected pairs of that batch: gathered when
 *                    n_sel <= rho_max * T * E, dense otherwise.  Both pairs of
 *                    kernels are enqueued and the pair not needed returns at once,
 *                    so there is no host synchronisation.  Batches whose up
 *                    projection is below 2e11 FLOP (about 150 us of tensor-core
 *                    time) always take the dense form: the gathered kernels'
 *                    fixed costs leave them little to win there, and the dense
 *                    kernel then keeps its overlap with the router.
 * group: experts per group, 0 = library default for the shape (a power of two
 * that divides E, group * expert_size a multiple of 16 and at most 256, 128 for
 * gated layers).  rho_max: crossover density of D2D_PATH_AUTO, negative =
 * library default for the shape.  Returns D2D_ERR_UNSUPPORTED when the shape
 * cannot take the gathered path (fp32 layers, expert sizes that are not a
 * multiple of 8) and it, or a group, was asked for.
 * With D2D_PATH_FUSED `group` sets the fused kernel's group (0 = the widest of
 * at most 128 neurons) and rho_max is ignored.  Under D2D_PATH_AUTO the fused
 * kernel is a third range below the gathered pair: it runs while
 * n_sel <= fused_rho_max * T * E (d2d_layer_set_fused_rho_max: negative =
 * library default for the shape, 0 = never; D2D_ERR_UNSUPPORTED for a positive
 * value on a shape the fused kernel cannot take: gated, fp32, d_ff < 2 d,
 * d < 128 or d > 4096). */
typedef enum { D2D_PATH_AUTO = 0, D2D_PATH_DENSE = 1, D2D_PATH_GATHER = 2, D2D_PATH_FUSED = 3 } d2d_expert_path;
D2D_API d2d_status d2d_layer_set_expert_path(d2d_layer *layer, d2d_expert_path path, int32_t group, double rho_max);
D2D_API d2d_status d2d_layer_set_fused_rho_max(d2d_layer *layer, double rho_max);
/* The fused kernel's group (0: the shape cannot take it) and the upper end of
 * its range under D2D_PATH_AUTO; either output pointer may be NULL. */
D2D_API d2d_status d2d_layer_get_fused(const d2d_layer *layer, int32_t *group, double *rho_max);
/* Current setting; any output pointer may be NULL.  *group is 0 when the shape
 * cannot take the gathered path, *rho_max is negative while the library default
 * is in force: that default depends on the batch size of each call (the
 * gathered kernels have a fixed cost that a small batch cannot amortise). */
D2D_API d2d_status d2d_layer_get_expert_path(const d2d_layer *layer, int32_t *path, int32_t *group, double *rho_max);
/* Which form of the expert step (D2D_PATH_DENSE, _GATHER or _FUSED) a call
 * with T tokens and n_sel selected pairs takes under the layer's current
 * setting: the rule the kernels evaluate on the device, evaluated on the host
 * (for bf16 batches above the decode sizes; reporting and tests). */
D2D_API d2d_status d2d_layer_expert_path_for(const d2d_layer *layer, int32_t T, int64_t n_sel, int32_t *path);

/* Clears the layer-owned device counters (the "last CTA" tickets, the tile and
 * sub-chunk counters of the expert kernels).  They reset themselves when a
 * call completes; a call that ended with D2D_ERR_TIMEOUT in the status word
 * may have left them non-zero, and the next call would then skip work.  Enqueue
 * this on the stream after such a call (it is a 1-2 KB memset). */
D2D_API d2d_status d2d_layer_reset_counters(d2d_layer *layer, void *stream);

/* Bytes of device workspace that any call on `layer` with up to max_tokens
 * tokens needs (256-byte aligned buffer).  Returns 0 for a NULL layer. */
D2D_API size_t d2d_workspace_bytes(const d2d_layer *layer, int32_t max_tokens);

/* Bytes of device workspace d2d_select_dynk / d2d_routing_from_mask need. */
D2D_API size_t d2d_select_workspace_bytes(int32_t T, int32_t E);

/* Router forward (Sec. 3.3): R[t,i] = | b_r2[i] + sum_j W_r2[i,j] relu(b_r1[j] + W_r1[j,:] x_t) |.
 * x: device [T, d] of desc.dtype.  R: device [T, E] float32 (always float32:
 * the selection rule is evaluated on these values).  Products accumulate in
 * float32.  ws: device workspace of at least d2d_workspace_bytes(layer, T). */
D2D_API d2d_status d2d_router_fwd(const d2d_layer *layer, const void *x, int32_t T, float *R,
                          void *ws, size_t ws_bytes, void *stream);

/* Dynamic-k selection and routing metadata (Eq. 4; Listing 1's per-expert
 * token lists and counts).  R: device [T, E] float32, expected finite and
 * non-negative.  For every token: m = max_i R[t,i]; thr = tau*m rounded once to
 * float32; expert i is kept iff R[t,i] >= thr (ties kept; an all-zero row keeps
 * every expert).  A token whose row holds a NaN or an infinity keeps every
 * expert and sets *status = D2D_ERR_NONFINITE.  Inside an expert's list tokens
 * are in ascending order, which makes every output unique (bit-exact
 * comparable).  If n_sel > perm_capacity, perm/tok_exp are truncated, the other
 * outputs are complete and *status = D2D_ERR_CAPACITY.  tau must lie in [0,1]. */
D2D_API d2d_status d2d_select_dynk(const float *R, int32_t T, int32_t E, float tau, d2d_routing *out,
                           void *ws, size_t ws_bytes, void *stream);

/* Static top-k selection (Sec. 3.3 notes that a router trained by regression
 * on the experts' output norms can also drive a fixed top-k rule): keeps the kk largest scores of each token, equal scores in
 * order of the lower expert index, then builds the same metadata. */
D2D_API d2d_status d2d_select_topk(const float *R, int32_t T, int32_t E, int32_t kk, d2d_routing *out,
                           void *ws, size_t ws_bytes, void *stream);

/* Routing metadata from a caller-supplied mask (the latency protocol of
 * Sec. 4.4 overrides the gating decisions with Bernoulli samples).
 * out->mask is the INPUT here (device, same layout; bits at positions >= E
 * must be zero); k, counts, offsets, perm, n_sel (and the dual) are written. */
D2D_API d2d_status d2d_routing_from_mask(int32_t T, int32_t E, d2d_routing *out,
                                 void *ws, size_t ws_bytes, void *stream);

/* d2d_select_dynk for callers that may not allocate device memory.  (The paper
 * has no counterpart; this is a deployment convenience.)
 * Some integrations run the layer from a context in which cudaMalloc is off
 * limits: a plug-in whose enqueue hook must not allocate, a serving loop whose
 * memory pool was fixed at start-up, code that runs after the framework has
 * handed all device memory to its own allocator.  Such a caller cannot obtain
 * the workspace d2d_select_dynk asks for, so this variant keeps the scratch it
 * needs in a fixed 512 KiB array inside the library's device image (every GPU
 * that loads the library holds it until the process exits).  The call itself
 * allocates nothing, on the host or the device, and frees nothing.
 *   - Same inputs, outputs, rule and error reporting as d2d_select_dynk; the
 *     caller still passes R and the routing buffers.
 *   - Limit: 64 + ceil(T / 256) * E <= 131072 (for example 16,000 tokens at
 *     2,048 experts, or 87,000 tokens at 384 experts); beyond it the call
 *     returns D2D_ERR_UNSUPPORTED and enqueues nothing.
 *   - The first call on each device looks up the array's device address (once,
 *     with that device current).  Make that first call outside any stream
 *     capture.
 *   - All calls on one device share the array, so two calls whose kernels can
 *     overlap on the GPU (different streams) race; serialise them.  The array
 *     keeps the previous call's contents: the one word that must start at
 *     zero is cleared by every call, every other entry is overwritten before
 *     it is read. */
D2D_API d2d_status d2d_select_dynk_static(const float *R, int32_t T, int32_t E, float tau, d2d_routing *out,
                                          void *stream);

/* Expert FFN and combine (Sec. 3.2, 3.4; App. G for the gated form):
 *   y[t,:] = b2 + sum over kept experts e of  W2[:, e-block] * h_e(x_t),
 *   h_e = A(W1[e-block,:] x_t + b1[e-block])           (gated: A(W_gate x) * (W1 x + b1)).
 * No router-score weighting (G is binary).  A token that keeps no expert gets
 * y = b2.  x, y: device [T, d] of desc.dtype; sums accumulate in float32; the
 * summation order over experts is not fixed, so y matches a reference within a
 * tolerance, not bit for bit.  `routing` must describe these T tokens. */
D2D_API d2d_status d2d_moe_ffn_fwd(const d2d_layer *layer, const void *x, int32_t T, const d2d_routing *routing,
                           void *y, void *ws, size_t ws_bytes, void *stream);

/* The two halves of the tensor-core expert step, exposed so that each can be
 * called, checked and timed on its own (bf16 layers only; other layers return
 * D2D_ERR_UNSUPPORTED).
 * d2d_expert_up_fwd (Sec. 3.2; gated form App. G):
 *   H[t, n] = G[t, n / s] ? A(W1[n,:] x_t + b1[n]) : 0        (gated: A(W_gate x)_n * (W1 x + b1)_n)
 * for every neuron n of the original FFN: the expert up projections of all
 * kept (token, expert) pairs as one dense contraction with the selection
 * applied as a mask.  x: device [T, d]; H: device [T, d_ff] bf16 (caller's).
 * d2d_expert_up_gather_fwd: the gathered kernel (D2D_PATH_GATHER with the
 * layer's group size), whatever path the layer is set to.  It writes ONLY the
 * cells H[t, group columns] of kept (token, group) pairs -- with the same
 * values d2d_expert_up_fwd writes there -- and leaves every other cell of H
 * untouched; D2D_ERR_UNSUPPORTED for shapes the gathered path cannot take.
 * d2d_expert_down_masked_fwd: y = (G * H) W2^T + b2 with the selection applied
 * while H is read (cells of unkept (token, expert) pairs are never read), the
 * down projection that follows the gathered kernel; valid for any H whose kept
 * cells hold the hidden activations.  Needs routing->mask and ->status only.
 * d2d_expert_down_fwd (Sec. 3.2, 3.4): y = H W2^T + b2, which is
 * b2 + sum over kept experts of W2[:, blk] h_blk.  y: device [T, d] bf16;
 * status: device status word (receives D2D_ERR_TIMEOUT), may be NULL. */
D2D_API d2d_status d2d_expert_up_fwd(const d2d_layer *layer, const void *x, int32_t T, const d2d_routing *routing,
                                     void *H, void *stream);
D2D_API d2d_status d2d_expert_up_gather_fwd(const d2d_layer *layer, const void *x, int32_t T, const d2d_routing *routing,
                                            void *H, void *stream);
D2D_API d2d_status d2d_expert_down_masked_fwd(const d2d_layer *layer, const void *H, int32_t T, const d2d_routing *routing,
                                              void *y, void *stream);
D2D_API d2d_status d2d_expert_down_fwd(const d2d_layer *layer, const void *H, int32_t T, void *y, int32_t *status,
                                       void *stream);

/* Test aid for the library's failure handling (no counterpart in the paper).
 * kind = 1: the NEXT d2d_expert_up_fwd call launches its kernel with one
 * operand load left out in one CTA, so that the bounded waits inside that CTA
 * run out (about a second): the kernel records D2D_ERR_TIMEOUT in the status
 * word, every warp role reaches the final barrier, tensor memory is freed and
 * the kernel returns normally -- nothing traps and no wait is unbounded.  H is
 * incomplete after such a call.  kind = 0 clears a pending request.  Follow a
 * timed-out call with d2d_layer_reset_counters before the layer is used again. */
D2D_API d2d_status d2d_test_inject_fault(int32_t kind);

/* The whole layer with no host synchronisation in between:
 * router_fwd -> select_dynk -> moe_ffn_fwd (Sec. 3.2-3.4).  R_out: optional
 * device [T,E] float32 output of the router scores; with NULL the scores may
 * never reach memory (for bf16 batches of 5 or more tokens the router kernel
 * thresholds them on chip).  `routing` supplies the metadata buffers (they
 * are outputs): mask, k and status are required; the per-expert lists
 * (counts, offsets, perm, n_sel and the dual) may be NULL as a set, in which
 * case they are not built -- allowed where the expert kernels read only the
 * mask (bf16 batches of more than 64 tokens; from 5 tokens with d_h = 128 and
 * E <= 256; small float32 problems), D2D_ERR_INVALID_ARG elsewhere.  Work is enqueued on `stream`; the per-expert
 * metadata may be built on a stream the layer owns, joined back into `stream`
 * before the call's last operation, so everything the call writes is ordered
 * before whatever the caller enqueues on `stream` next.  The layer object
 * holds that side stream, two events and the self-resetting tickets of the
 * decode kernels: calls on ONE layer object must not overlap in time (use one
 * layer object per stream for concurrent streams).  On `stream` the up
 * projection may start before the router has finished (programmatic dependent
 * launch); it reads only x and the weights until the router has completed. */
D2D_API d2d_status d2d_layer_fwd(const d2d_layer *layer, const void *x, int32_t T, float tau, void *y,
                         float *R_out, d2d_routing *routing, void *ws, size_t ws_bytes, void *stream);

/* Host-buffer convenience: the same layer call, but x and y are HOST pointers
 * ([T,d] of desc.dtype).  The call copies x to the device, runs the layer,
 * copies y back and synchronises `stream`; all device memory it needs comes
 * from `ws` (device, at least d2d_layer_fwd_host_workspace_bytes bytes).
 * Batches of 8192 tokens or more are cut into four chunks of 3/16, 5/16, 5/16
 * and 3/16 of the tokens (the call then takes about the copy-in of the first
 * chunk + the layer on all of them + the copy-out of the last) and pipelined over
 * two copy streams the layer owns (copy in / layer / copy out overlap; tokens
 * are independent, so the result is the same); this needs page-locked host
 * buffers to be effective.  Returns the data-dependent status as well
 * (D2D_ERR_NONFINITE, D2D_ERR_TIMEOUT), read back after the synchronisation. */
D2D_API size_t d2d_layer_fwd_host_workspace_bytes(const d2d_layer *layer, int32_t max_tokens);
D2D_API d2d_status d2d_layer_fwd_host(const d2d_layer *layer, const void *x_host, int32_t T, float tau, void *y_host,
                              void *ws, size_t ws_bytes, void *stream);

/* Layer groups (Sec. 3.5: every projection matrix of the attention layer is
 * replaced by its own MoE layer, so a converted block has four MoE layers in
 * the attention and one in the FFN).  The Q, K and V projections read the same
 * token rows: a group holds n_layers (1..4) layers of ONE shape (equal desc)
 * and runs them on a shared input as one launch sequence.  Each layer keeps
 * its own router, its own threshold rule (max over ITS experts, Eq. 4) and its
 * own output; the result equals n_layers separate d2d_layer_fwd calls.
 *   layers   : host array of layer handles; the group does not own them and
 *              they must outlive it; a layer may appear once.
 *   x        : device [T, d] of desc.dtype, shared by all layers.
 *   y        : device [n_layers, T, d] (layer l's output at y + l*T*d elements;
 *              T*d*sizeof(elem) must be a multiple of 16).
 *   routing  : host array of n_layers d2d_routing (outputs, all required as
 *              in d2d_layer_fwd); routing[l] describes layer l.
 *   ws       : device workspace of at least d2d_group_workspace_bytes bytes.
 * bf16, not gated, d_h = 128, E a multiple of 32 and at most 256, d_ff a
 * multiple of 64: the group owns stacked copies of the weights and the routers
 * run as one grid, the up projections as one GEMM and the down projections as
 * one batched GEMM (T of 5 or more); for T <= 4 (fp32: T <= 8) of any shape
 * the decode kernels serve all layers in two launches.  Other shapes run the
 * layers one after the other.  Device status: timeouts of the merged GEMMs
 * are reported in routing[0].status.  Like a layer, a group (and its layers)
 * serves one call at a time. */
typedef struct d2d_group d2d_group;
D2D_API d2d_status d2d_group_create(d2d_layer *const *layers, int32_t n_layers, void *stream, d2d_group **out);
D2D_API d2d_status d2d_group_destroy(d2d_group *group);
D2D_API size_t d2d_group_workspace_bytes(const d2d_group *group, int32_t max_tokens);
D2D_API d2d_status d2d_group_fwd(const d2d_group *group, const void *x, int32_t T, float tau, void *y,
                                 d2d_routing *routing, void *ws, size_t ws_bytes, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* D2D_H_ */
