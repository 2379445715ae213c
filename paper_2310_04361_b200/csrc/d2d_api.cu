// Host side of the C ABI declared in include/d2d.h: argument validation, weight packing,
// workspace carving and kernel dispatch.  No computation happens on the host.
#include <limits.h>
#include <math.h>
#include <new>
#include <string.h>

#include "d2d_common.cuh"
#include <stdlib.h>
#include "gemm_tc.cuh"
#include "moe_gather.cuh"

bool d2d_token_path_supports(const d2d_layer_desc &D);
d2d_status d2d_launch_moe_ffn_token(const d2d_layer *L, const void *x, int T, const d2d_routing *r, void *y,
                                    cudaStream_t st);

unsigned long long d2d_launch_counter = 0;
static int g_test_fault = 0;       // d2d_test_inject_fault: consumed by the next d2d_expert_up_fwd

namespace {

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool has_lists(const d2d_routing *r) { return r->counts && r->offsets && r->perm && r->n_sel; }

// lists_optional: the per-expert lists (counts, offsets, perm, n_sel) may be absent as a set (d2d_layer_fwd then
// does not build them); mask, k and status are always required
bool routing_ok(const d2d_routing *r, bool lists_optional)
{
    if (!r || !r->mask || !r->k || !r->status) return false;
    const bool none = !r->counts && !r->offsets && !r->perm && !r->n_sel && !r->tok_off && !r->tok_exp;
    if (lists_optional && none) return true;
    if (!has_lists(r)) return false;
    if ((r->tok_off == nullptr) != (r->tok_exp == nullptr)) return false;
    return r->perm_capacity >= 0;
}

// Workspace layout of the layer-level calls: [ u: T*d_h f32 | R: T*E f32 | select scratch | ffn scratch ]
struct ws_layout {
    size_t u_off, r_off, sel_off, ffn_off, total;
};

ws_layout layout_for(const d2d_layer *L, int T)
{
    ws_layout w;
    const size_t Tn = (size_t)(T > 0 ? T : 1);
    size_t off = 0;
    w.u_off = off;
    off += 256 + d2d_align_up(Tn * (size_t)L->desc.d_h * sizeof(float), 256);   // ticket area + hidden activations
    w.r_off = off;
    off += d2d_align_up(Tn * (size_t)L->desc.n_experts * sizeof(float), 256);
    w.sel_off = off;
    off += d2d_select_ws_bytes((int)Tn, L->desc.n_experts);
    w.ffn_off = off;
    off += d2d_moe_ffn_ws_bytes(L, (int)Tn);
    w.total = off;
    return w;
}

}  // namespace

// Up to this many tokens a bf16 layer takes the decode kernels.  Measured (us per layer call, decode kernels /
// tensor-core path): GPT-2-medium-shaped FFN (64 KB of weights per expert) T = 3: 31 / 39, T = 4: 33 / 39, T = 5:
// 41 / 40, T = 8: 43 / 39; Llama-shaped layer (786 KB per expert) T = 1: 84 / 129, T = 2: 108 / 133, T = 3: 221 / 133,
// T = 4: 229 / 127.  So 4 tokens for small experts, 2 for large ones; D2D_DECODE_MAX_TOKENS overrides both.
int d2d_decode_max_tokens(const d2d_layer_desc &D)
{
    static const int v = [] {
        const char *e = getenv("D2D_DECODE_MAX_TOKENS");
        const int n = e ? atoi(e) : -1;
        return n > 8 ? 8 : n;
    }();
    if (v >= 0) return v;
    const size_t expert_bytes = (size_t)(D.gated ? 3 : 2) * D.expert_size * D.d * 2;
    return expert_bytes > ((size_t)256 << 10) ? 2 : 4;
}

static bool use_dense_masked(const d2d_layer *L, int T)
{
    return L->desc.dtype == D2D_BF16 && T > d2d_decode_max_tokens(L->desc) && L->desc.d_ff % 8 == 0 && d2d_gemm_tc_available();
}

// Up to this many tokens the expert-per-CTA kernel (each kept expert's slice read once) is used.

static bool use_small_ffn(const d2d_layer *L, int T)
{
    const int lim = L->desc.dtype == D2D_BF16 ? d2d_decode_max_tokens(L->desc) : 8;      // fp32 layers have no tensor-core path
    return T <= lim && d2d_small_ffn_supports(L->desc);
}

size_t d2d_moe_ffn_ws_bytes(const d2d_layer *L, int T)
{
    size_t need = 256;
    if (use_small_ffn(L, T)) need = d2d_small_ffn_ws_bytes(L, T);
    // hidden activations H [T, d_ff] bf16 of the dense-masked path
    if (L->desc.dtype == D2D_BF16 && T > d2d_decode_max_tokens(L->desc)) {
        size_t h = d2d_align_up((size_t)T * L->desc.d_ff * 2, 256);
        if (d2d_gemm_tc_splits(T, L->desc.d, L->desc.d_ff) > 1) h += d2d_align_up((size_t)T * L->desc.d * 4, 256);   // split-K partial sums
        if (h > need) need = h;
    }
    return need;
}

// Density up to which the gathered pair beats the masked dense pair for this shape and batch size: the default
// crossover of the automatic choice.  Measured on B200: the gathered kernel is bound by the rate at which token rows
// can be copied into the A stages (about the same time per 128 x 64 tile of gathered rows whatever the MMA width), so
// with full-width groups a gathered row costs about 1.2 x a dense one, and the kernel has a fixed part (the scan of the
// mask, a ragged tile per group visit) worth about five tiles per CTA.  Against a dense up projection of
// T / 128 x Nd tiles (Nd = 256-column tiles across d_ff) on S SMs that fixed part is T0 = 5 * 128 * 1.2 * S / Nd
// tokens' worth of dense time, so the pair wins while the fraction of kept (token, group) pairs
//     u = 1 - (1 - rho)^g  <  U - T0 / T,
// U = 0.85 for 256 MMA columns (less for narrower groups).  Checked against measured crossovers: Llama-shaped
// layer u = 0.70 at 8192 tokens, 0.55 at 4096; paper's latency shape 0.7 at 50432 tokens (357 against 374 us at rho = 0.4, 387 against 381 us at 0.5); ViT-shaped 0.5 at
// 25216; never for the BERT-shaped layer at 4096 tokens.
int d2d_tc_sm_count();      // gemm_tc.cu

static const double kAutoMinUpFlop = 2e11;      // smallest up projection for which the automatic choice is made

static double default_gather_rho_max(const d2d_layer_desc &D, int g, int T)
{
    if (g <= 0 || T <= 0) return -1.0;
    const int n_mma = g * D.expert_size * (D.gated ? 2 : 1);
    double U = n_mma >= 256 ? 0.85 : n_mma >= 192 ? 0.64 : n_mma >= 128 ? 0.43 : 0.25;
    const double nd = ceil((double)D.d_ff * (D.gated ? 2.0 : 1.0) / 256.0);
    const double T0 = 5.0 * 128.0 * 1.2 * (double)d2d_tc_sm_count() / nd;
    const double u_max = U - T0 / (double)T;
    if (u_max <= 0.0) return 0.0;
    return 1.0 - pow(1.0 - u_max, 1.0 / g);
}

// Density up to which the fused gathered kernel beats both pairs.  Its merge moves 4 d bytes of vector reductions per
// kept (token, group) pair through each SM's path to L2, next to the token and weight rows coming in, and its float32
// accumulator is written once and read once more than the other paths' output: measured on B200 (d = 768, 128-neuron
// groups, 50432 tokens: 141 / 151 / 174 / 244 us at 1 / 2 / 5 / 10 % of the pairs kept, gathered pair 217 / 225 / 231 /
// 248 us) it wins while at most about 8 % of the (token, group) pairs are kept.
static double default_fused_rho_max(int g)
{
    if (g <= 0) return 0.0;
    return 1.0 - pow(1.0 - 0.08, 1.0 / g);
}

// Expert step of bf16 batches above the decode sizes, on the tensor cores.
//   up projection    two kernels that compute the same H = G * A(x W1^T + b1):
//     masked dense   one GEMM over all of d_ff, the selection applied as a mask in the epilogue; its time does not
//                    depend on the selection (every expert is kept by some token of a 128-token tile)
//     gathered       per group of adjacent experts, a contraction over the tokens that keep the group (moe_gather.cu);
//                    its time is proportional to the number of (token, group) pairs
//   down projection  y = H W2^T + b2 as a dense GEMM: exactly b2 + the sum over kept experts, since the h of an expert
//                    the token did not keep is zero (written as zero by the masked dense kernel, or zero-filled from
//                    the mask while H is staged when the gathered kernel, which writes only kept cells, may have run)
// Which up projection runs is decided per call from the number of selected pairs of THIS batch.  D2D_PATH_AUTO
// launches both kernels with complementary rules on a device word (n_sel) that is valid once the preceding kernel of
// the stream has completed; the one that is not needed returns at once, so no host synchronisation is involved.
// up_counter (optional): a zeroed device counter; its presence also states that the kernel launched just before
// on this stream is the router, which writes only the mask (and R, k), so that a forced masked dense up projection
// may overlap it with its main loops and draw its tiles dynamically.
static d2d_status launch_tc_experts(const d2d_layer *L, const void *x, int T, const d2d_routing *r, void *y,
                                    void *ws, cudaStream_t st, int *up_counter, const int32_t *n_sel)
{
    const d2d_layer_desc &D = L->desc;
    int path = L->expert_path;
    if (L->gather_group <= 0) path = D2D_PATH_DENSE;
    // The automatic choice costs a few launches that return at once and the overlap of the router with the masked dense
    // kernel's main loops (measured on the ViT-shaped layer, 1.2e11 FLOP: 241 us against 224 us at every density, while
    // the gathered paths win there only below rho = 0.03): it is made only for problems whose up projection takes long
    // enough (2e11 FLOP, about 150 us of tensor-core time) that this is noise.
    const double up_flop = 2.0 * (double)T * D.d * D.d_ff * (D.gated ? 2.0 : 1.0);
    if (path == D2D_PATH_AUTO && (up_flop < kAutoMinUpFlop || !n_sel)) path = D2D_PATH_DENSE;
    const double rho_max = L->gather_rho_max >= 0.0 ? L->gather_rho_max : default_gather_rho_max(D, L->gather_group, T);
    long long n_sel_max = (long long)(rho_max * (double)T * (double)D.n_experts);
    d2d_status rc;
    // Fused gathered step (plain layers): up projection, activation, down projection and the merge in one kernel whose
    // time is proportional to the kept (token, group) pairs; the float32 accumulator takes the place of H.
    long long n_sel_fused = -1;
    if (L->fused_group > 0 && (path == D2D_PATH_FUSED || (path == D2D_PATH_AUTO && L->fused_rho_max > 0.0))) {
        d2d_gather_args fa = {};
        fa.x = x; fa.w1 = L->w1; fa.b1 = L->b1; fa.mask = r->mask;
        fa.T = T; fa.d = D.d; fa.d_ff = D.d_ff; fa.n_experts = D.n_experts; fa.s = D.expert_size; fa.g = L->fused_group;
        fa.act = D.act; fa.status = r->status; fa.ctr = L->gather_ctr;
        if (path == D2D_PATH_AUTO) {
            // three ranges of n_sel: (.., fused] fused kernel, (fused, max] gathered pair, (max, ..) dense pair
            n_sel_fused = (long long)(L->fused_rho_max * (double)T * (double)D.n_experts);
            if (n_sel_max < n_sel_fused) n_sel_max = n_sel_fused;
            fa.n_sel = n_sel; fa.n_sel_min = -1; fa.n_sel_max = n_sel_fused;
        }
        rc = d2d_moe_gather_ffn(fa, (float *)ws, y, L->w2, L->b2, st);
        if (rc != D2D_OK || path == D2D_PATH_FUSED) return rc;
    } else if (path == D2D_PATH_FUSED) {
        return D2D_ERR_UNSUPPORTED;
    }
    if (path != D2D_PATH_GATHER) {
        d2d_gemm_args up = {};
        const bool forced = path == D2D_PATH_DENSE;
        up.tile_counter = forced ? up_counter : nullptr;
        up.pdl_late_wait = forced && up_counter != nullptr;
        up.n_sel = forced ? nullptr : n_sel; up.n_sel_max = n_sel_max;
        up.a = x; up.b = L->w1; up.b_gate = D.gated ? L->w_gate : nullptr; up.b_cat = L->w1g; up.b_cat_block = 128; up.bias = L->b1; up.out = ws;
        up.M = T; up.N = D.d_ff; up.K = D.d; up.epilogue = D2D_EPI_UP_MASKED; up.act = D.act;
        up.mask = r->mask; up.mask_words = (D.n_experts + 31) / 32; up.expert_size = D.expert_size; up.status = r->status;
        rc = d2d_gemm_tc(up, st);
        if (rc != D2D_OK) return rc;
    }
    // Wide layers: the cells the gathered kernel leaves alone are zero-filled, so that the TMA-fed dense down projection
    // can follow whichever up projection ran; otherwise the down projection that applies the selection while it stages
    // H follows the gathered kernel.
    const bool zero_fill = path != D2D_PATH_DENSE && D.d >= 2048;
    if (path != D2D_PATH_DENSE) {
        const long long hi = path == D2D_PATH_AUTO ? n_sel_max : LLONG_MAX;
        if (zero_fill) {
            // on the layer's side stream: the fill and the gathered kernel write disjoint cells, and its small CTAs fit
            // beside the persistent ones; joined before the down projection
            if (cudaEventRecord(L->ev_fill_fork, st) != cudaSuccess || cudaStreamWaitEvent(L->side_stream, L->ev_fill_fork, 0) != cudaSuccess)
                return D2D_ERR_CUDA;
            rc = d2d_moe_zero_unkept(ws, r->mask, T, D.d_ff, D.n_experts, D.expert_size, L->gather_group, n_sel, n_sel_fused, hi,
                                     L->side_stream);
            if (rc != D2D_OK) return rc;
            if (cudaEventRecord(L->ev_fill_join, L->side_stream) != cudaSuccess) return D2D_ERR_CUDA;
        }
        d2d_gather_args ga = {};
        ga.x = x; ga.w1 = L->w1; ga.w_gate = D.gated ? L->w_gate : nullptr; ga.b1 = L->b1; ga.mask = r->mask; ga.H = ws;
        ga.T = T; ga.d = D.d; ga.d_ff = D.d_ff; ga.n_experts = D.n_experts; ga.s = D.expert_size; ga.g = L->gather_group;
        ga.act = D.act; ga.status = r->status; ga.ctr = L->gather_ctr;
        ga.n_sel = n_sel; ga.n_sel_min = n_sel_fused; ga.n_sel_max = hi;
        rc = d2d_moe_gather_up(ga, st);
        if (rc != D2D_OK) return rc;
    }
    if (path != D2D_PATH_DENSE && !zero_fill) {
        rc = d2d_moe_down_masked(D, ws, r->mask, L->w2, L->b2, y, T, r->status, st, path == D2D_PATH_AUTO ? n_sel : nullptr, n_sel_fused, n_sel_max);
        if (rc != D2D_OK || path == D2D_PATH_GATHER) return rc;
    }
    if (zero_fill && cudaStreamWaitEvent(st, L->ev_fill_join, 0) != cudaSuccess) return D2D_ERR_CUDA;
    d2d_gemm_args dn = {};
    dn.a = ws; dn.b = L->w2; dn.bias = L->b2; dn.out = y;
    // after a zero fill this kernel serves the gathered range too: it only has to stay out of the fused kernel's range
    dn.n_sel = path == D2D_PATH_AUTO && (!zero_fill || n_sel_fused >= 0) ? n_sel : nullptr;
    dn.n_sel_max = zero_fill ? n_sel_fused : n_sel_max;
    dn.M = T; dn.N = D.d; dn.K = D.d_ff; dn.epilogue = D2D_EPI_BIAS_BF16; dn.status = r->status;
    // decode-sized batches: split K over the SMs, partial sums in the float32 scratch behind H
    dn.k_splits = d2d_gemm_tc_splits(T, D.d, D.d_ff);
    dn.partial = dn.k_splits > 1 ? (float *)((char *)ws + d2d_align_up((size_t)T * D.d_ff * 2, 256)) : nullptr;
    return d2d_gemm_tc(dn, st);
}

d2d_status d2d_launch_moe_ffn(const d2d_layer *L, const void *x, int T, const d2d_routing *r, void *y,
                              void *ws, size_t ws_bytes, cudaStream_t st, int *up_counter, int small_fused, const int32_t *n_sel)
{
    if (ws_bytes < d2d_moe_ffn_ws_bytes(L, T)) return D2D_ERR_WORKSPACE;
    if (use_small_ffn(L, T)) return has_lists(r) ? d2d_small_ffn(L, x, T, r, y, ws, st, small_fused) : D2D_ERR_INVALID_ARG;
    if (use_dense_masked(L, T)) return launch_tc_experts(L, x, T, r, y, ws, st, up_counter, n_sel ? n_sel : r->n_sel);
    return d2d_launch_moe_ffn_token(L, x, T, r, y, st);
}

extern "C" {

uint64_t d2d_launch_count(void) { return __atomic_load_n(&d2d_launch_counter, __ATOMIC_RELAXED); }

const char *d2d_status_str(d2d_status s)
{
    switch (s) {
    case D2D_OK: return "ok";
    case D2D_ERR_INVALID_ARG: return "invalid argument";
    case D2D_ERR_UNSUPPORTED: return "unsupported shape or option";
    case D2D_ERR_WORKSPACE: return "workspace too small";
    case D2D_ERR_CUDA: return "CUDA runtime or launch failure";
    case D2D_ERR_NONFINITE: return "non-finite router score";
    case D2D_ERR_TIMEOUT: return "bounded wait ran out inside a kernel";
    case D2D_ERR_CAPACITY: return "more selected pairs than perm_capacity";
    }
    return "unknown status";
}

// Gated bf16 layers: W1 and W_gate once more, interleaved in blocks of 128 rows (the gated up projection fetches both
// tiles with one TMA box).  Built from the layer's own packed copies (again after they were replaced by dequantised values).
static d2d_status build_gate_cat(d2d_layer *L, cudaStream_t st)
{
    const d2d_layer_desc &D = L->desc;
    const int cat_block = 128;
    const size_t cat_rows = (size_t)2 * cat_block * d2d_cdiv(D.d_ff, cat_block);
    const size_t row_b = (size_t)D.d * L->elem;
    char *cat = (char *)L->w1g;
    if (cudaMemsetAsync(cat, 0, cat_rows * row_b, st) != cudaSuccess) return D2D_ERR_CUDA;
    for (int r0 = 0, b = 0; r0 < D.d_ff; r0 += cat_block, ++b) {
        const size_t rows = (size_t)(D.d_ff - r0 < cat_block ? D.d_ff - r0 : cat_block);
        char *dst = cat + (size_t)b * 2 * cat_block * row_b;
        if (cudaMemcpyAsync(dst, (const char *)L->w1 + (size_t)r0 * row_b, rows * row_b, cudaMemcpyDeviceToDevice, st) != cudaSuccess ||
            cudaMemcpyAsync(dst + (size_t)cat_block * row_b, (const char *)L->w_gate + (size_t)r0 * row_b, rows * row_b,
                            cudaMemcpyDeviceToDevice, st) != cudaSuccess)
            return D2D_ERR_CUDA;
    }
    return D2D_OK;
}

d2d_status d2d_layer_create(const d2d_layer_desc *desc, const d2d_weights *w, void *stream, d2d_layer **out)
{
    if (out) *out = nullptr;
    if (!desc || !w || !out) return D2D_ERR_INVALID_ARG;
    const d2d_layer_desc &D = *desc;
    if (D.d <= 0 || D.d_ff <= 0 || D.n_experts <= 0 || D.expert_size <= 0 || D.d_h <= 0) return D2D_ERR_INVALID_ARG;
    if ((int64_t)D.n_experts * D.expert_size != D.d_ff) return D2D_ERR_INVALID_ARG;
    if (D.dtype != D2D_F32 && D.dtype != D2D_BF16) return D2D_ERR_INVALID_ARG;
    if (D.act < D2D_ACT_RELU || D.act > D2D_ACT_SILU) return D2D_ERR_INVALID_ARG;
    if (D.d % 8 || D.d_h % 8) return D2D_ERR_INVALID_ARG;
    if (!w->w_r1 || !w->w_r2 || !w->w1 || !w->w2) return D2D_ERR_INVALID_ARG;
    if ((D.gated != 0) != (w->w_gate != nullptr)) return D2D_ERR_INVALID_ARG;
    if (!d2d_token_path_supports(D)) return D2D_ERR_UNSUPPORTED;

    int dev = 0, sms = 0;
    D2D_CUDA_TRY(cudaGetDevice(&dev));
    D2D_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));

    d2d_layer *L = new (std::nothrow) d2d_layer();
    if (!L) return D2D_ERR_CUDA;
    memset(L, 0, sizeof(*L));
    L->desc = D;
    L->elem = D.dtype == D2D_F32 ? 4 : 2;
    L->sm_count = sms;
    const size_t el = L->elem;
    const size_t n_wr1 = (size_t)D.d_h * D.d, n_wr2 = (size_t)D.n_experts * D.d_h, n_w = (size_t)D.d_ff * D.d;

    struct piece { void **dst; const void *src; size_t n; bool transpose; };
    piece pieces[] = {
        {&L->w_r1, w->w_r1, n_wr1, false}, {&L->b_r1, w->b_r1, (size_t)D.d_h, false},
        {&L->w_r2, w->w_r2, n_wr2, false}, {&L->b_r2, w->b_r2, (size_t)D.n_experts, false},
        {&L->w1, w->w1, n_w, false},       {&L->b1, w->b1, (size_t)D.d_ff, false},
        {&L->w_gate, w->w_gate, n_w, false}, {&L->w2t, w->w2, n_w, true},
        {&L->b2, w->b2, (size_t)D.d, false}, {&L->w2, w->w2, n_w, false},
    };
    size_t total = 256;                                   // the ticket words (see d2d_layer::tickets)
    L->gather_group = d2d_gather_group_for(D, 0);
    L->gather_rho_max = -1.0;                             // the default for the shape and the batch size of each call
    L->expert_path = D2D_PATH_AUTO;
    L->fused_group = d2d_gather_ffn_group_for(D);
    L->fused_rho_max = default_fused_rho_max(L->fused_group);
    L->gather_ctr_words = D.n_experts + 64;               // enough for any group size: E / g counters + the exit ticket
    const size_t ctr_off = total;
    total += d2d_align_up((size_t)L->gather_ctr_words * sizeof(int), 256);
    for (const piece &p : pieces)
        if (p.src) total += d2d_align_up(p.n * el, 256);
    // gated bf16 layers: W1 and W_gate once more, interleaved in blocks of 128 rows for the tensor-core up projection
    const int cat_block = 128;
    const size_t cat_rows = (size_t)2 * cat_block * d2d_cdiv(D.d_ff, cat_block);
    const bool want_cat = D.gated && D.dtype == D2D_BF16;
    const size_t cat_off = total;
    if (want_cat) total += d2d_align_up(cat_rows * D.d * el, 256);
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMalloc(&L->slab, total) != cudaSuccess) {
        delete L;
        return D2D_ERR_CUDA;
    }
    L->slab_bytes = total;
    L->tickets = (unsigned int *)L->slab;
    L->gather_ctr = (int *)((char *)L->slab + ctr_off);
    size_t off = ctr_off + d2d_align_up((size_t)L->gather_ctr_words * sizeof(int), 256);
    d2d_status rc = cudaMemsetAsync(L->slab, 0, off, st) == cudaSuccess ? D2D_OK : D2D_ERR_CUDA;
    for (const piece &p : pieces) {
        if (!p.src || rc != D2D_OK) continue;
        void *dst = (char *)L->slab + off;
        off += d2d_align_up(p.n * el, 256);
        *p.dst = dst;
        if (p.transpose) {
            rc = d2d_launch_transpose(p.src, dst, D.d, D.d_ff, el, st);
        } else if (cudaMemcpyAsync(dst, p.src, p.n * el, cudaMemcpyDeviceToDevice, st) != cudaSuccess) {
            rc = D2D_ERR_CUDA;
        }
        if (rc != D2D_OK) break;
    }
    if (rc == D2D_OK && want_cat) {
        L->w1g = (char *)L->slab + cat_off;
        rc = build_gate_cat(L, st);
    }
    if (rc == D2D_OK && cudaStreamSynchronize(st) != cudaSuccess) rc = D2D_ERR_CUDA;
    if (rc == D2D_OK && (cudaStreamCreateWithFlags(&L->side_stream, cudaStreamNonBlocking) != cudaSuccess ||
                         cudaEventCreateWithFlags(&L->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
                         cudaEventCreateWithFlags(&L->ev_join, cudaEventDisableTiming) != cudaSuccess ||
                         cudaEventCreateWithFlags(&L->ev_fill_fork, cudaEventDisableTiming) != cudaSuccess ||
                         cudaEventCreateWithFlags(&L->ev_fill_join, cudaEventDisableTiming) != cudaSuccess))
        rc = D2D_ERR_CUDA;
    if (rc == D2D_OK) {
        bool ok = cudaStreamCreateWithFlags(&L->copy_in, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&L->copy_out, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaEventCreateWithFlags(&L->ev_begin, cudaEventDisableTiming) == cudaSuccess &&
                  cudaEventCreateWithFlags(&L->ev_end, cudaEventDisableTiming) == cudaSuccess;
        for (int c = 0; c < d2d_layer::kHostChunks && ok; ++c)
            ok = cudaEventCreateWithFlags(&L->ev_in[c], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&L->ev_done[c], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) rc = D2D_ERR_CUDA;
    }
    if (rc != D2D_OK) {
        d2d_layer_destroy(L);
        return rc;
    }
    *out = L;
    return D2D_OK;
}

d2d_status d2d_layer_destroy(d2d_layer *layer)
{
    if (!layer) return D2D_OK;
    if (layer->ev_join) cudaEventDestroy(layer->ev_join);
    if (layer->ev_fill_fork) cudaEventDestroy(layer->ev_fill_fork);
    if (layer->ev_fill_join) cudaEventDestroy(layer->ev_fill_join);
    if (layer->ev_fork) cudaEventDestroy(layer->ev_fork);
    if (layer->side_stream) cudaStreamDestroy(layer->side_stream);
    for (int c = 0; c < d2d_layer::kHostChunks; ++c) {
        if (layer->ev_in[c]) cudaEventDestroy(layer->ev_in[c]);
        if (layer->ev_done[c]) cudaEventDestroy(layer->ev_done[c]);
    }
    if (layer->ev_begin) cudaEventDestroy(layer->ev_begin);
    if (layer->ev_end) cudaEventDestroy(layer->ev_end);
    if (layer->copy_in) cudaStreamDestroy(layer->copy_in);
    if (layer->copy_out) cudaStreamDestroy(layer->copy_out);
    if (layer->q_slab) cudaFree(layer->q_slab);
    cudaError_t e = cudaFree(layer->slab);
    delete layer;
    return e == cudaSuccess ? D2D_OK : D2D_ERR_CUDA;
}

d2d_status d2d_layer_create_fp8(const d2d_layer_desc *desc, const d2d_weights *w, void *stream, d2d_layer **out)
{
    if (out) *out = nullptr;
    if (!desc || desc->dtype != D2D_BF16) return D2D_ERR_UNSUPPORTED;
    if (desc->d % 16 || ((int64_t)desc->expert_size * desc->d) % 16) return D2D_ERR_UNSUPPORTED;   // 16-byte pieces of codes
    d2d_layer *L = nullptr;
    d2d_status rc = d2d_layer_create(desc, w, stream, &L);
    if (rc != D2D_OK) return rc;
    const d2d_layer_desc &D = L->desc;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t n_w = (size_t)D.d_ff * D.d, n_mat = D.gated ? 3 : 2;
    const size_t codes_b = d2d_align_up(n_w, 256), exps_b = d2d_align_up((size_t)D.n_experts * sizeof(int32_t), 256);
    if (cudaMalloc(&L->q_slab, n_mat * (codes_b + exps_b)) != cudaSuccess) {
        d2d_layer_destroy(L);
        return D2D_ERR_CUDA;
    }
    char *q = (char *)L->q_slab;
    L->q_w1 = (uint8_t *)q; L->q_k1 = (int32_t *)(q + codes_b); q += codes_b + exps_b;
    L->q_w2t = (uint8_t *)q; L->q_k2 = (int32_t *)(q + codes_b); q += codes_b + exps_b;
    if (D.gated) { L->q_wg = (uint8_t *)q; L->q_kg = (int32_t *)(q + codes_b); }
    const int per = D.expert_size * D.d;
    // the packed bf16 copies are replaced by the dequantised values, so every path of the layer computes with them
    rc = d2d_quantize_experts_e4m3(L->w1, L->q_w1, L->q_k1, D.n_experts, per, st);
    if (rc == D2D_OK) rc = d2d_quantize_experts_e4m3(L->w2t, L->q_w2t, L->q_k2, D.n_experts, per, st);
    if (rc == D2D_OK && D.gated) rc = d2d_quantize_experts_e4m3(L->w_gate, L->q_wg, L->q_kg, D.n_experts, per, st);
    if (rc == D2D_OK) rc = d2d_launch_transpose(L->w2t, L->w2, D.d_ff, D.d, L->elem, st);      // W2 [d, d_ff] from the transposed copy
    if (rc == D2D_OK && L->w1g) rc = build_gate_cat(L, st);
    if (rc == D2D_OK && cudaStreamSynchronize(st) != cudaSuccess) rc = D2D_ERR_CUDA;
    if (rc != D2D_OK) {
        d2d_layer_destroy(L);
        return rc;
    }
    *out = L;
    return D2D_OK;
}

d2d_status d2d_layer_get_fp8(const d2d_layer *layer, int32_t which, uint8_t *codes, int32_t *exps, void *stream)
{
    if (!layer || which < 0 || which > 2 || (!codes && !exps)) return D2D_ERR_INVALID_ARG;
    const uint8_t *c = which == 0 ? layer->q_w1 : which == 1 ? layer->q_wg : layer->q_w2t;
    const int32_t *k = which == 0 ? layer->q_k1 : which == 1 ? layer->q_kg : layer->q_k2;
    if (!c || !k) return D2D_ERR_UNSUPPORTED;
    const d2d_layer_desc &D = layer->desc;
    cudaStream_t st = (cudaStream_t)stream;
    if (codes && cudaMemcpyAsync(codes, c, (size_t)D.d_ff * D.d, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return D2D_ERR_CUDA;
    if (exps && cudaMemcpyAsync(exps, k, (size_t)D.n_experts * sizeof(int32_t), cudaMemcpyDeviceToDevice, st) != cudaSuccess) return D2D_ERR_CUDA;
    return D2D_OK;
}

d2d_status d2d_layer_set_expert_path(d2d_layer *layer, d2d_expert_path path, int32_t group, double rho_max)
{
    if (!layer || path < D2D_PATH_AUTO || path > D2D_PATH_FUSED || group < 0) return D2D_ERR_INVALID_ARG;
    if (path == D2D_PATH_FUSED) {
        // the group size applies to the fused kernel, whose groups hold at most 128 neurons
        const d2d_layer_desc &D = layer->desc;
        int g = d2d_gather_ffn_group_for(D);
        if (g <= 0) return D2D_ERR_UNSUPPORTED;
        if (group > 0) {
            const int gs = group * D.expert_size;
            if ((group & (group - 1)) || group > 32 || D.n_experts % group || gs % 16 || gs > 128) return D2D_ERR_UNSUPPORTED;
            g = group;
        }
        layer->fused_group = g;
        layer->expert_path = path;
        return D2D_OK;
    }
    const int g = d2d_gather_group_for(layer->desc, group);
    if (g <= 0 && (path == D2D_PATH_GATHER || group > 0)) return D2D_ERR_UNSUPPORTED;
    layer->gather_group = g;
    layer->expert_path = path;
    layer->gather_rho_max = rho_max >= 0.0 ? (rho_max > 1.0 ? 1.0 : rho_max) : -1.0;
    return D2D_OK;
}

d2d_status d2d_layer_set_fused_rho_max(d2d_layer *layer, double rho_max)
{
    if (!layer) return D2D_ERR_INVALID_ARG;
    if (layer->fused_group <= 0) return rho_max > 0.0 ? D2D_ERR_UNSUPPORTED : D2D_OK;
    layer->fused_rho_max = rho_max >= 0.0 ? (rho_max > 1.0 ? 1.0 : rho_max) : default_fused_rho_max(layer->fused_group);
    return D2D_OK;
}

d2d_status d2d_layer_expert_path_for(const d2d_layer *layer, int32_t T, int64_t n_sel, int32_t *path)
{
    if (!layer || !path || T <= 0 || n_sel < 0) return D2D_ERR_INVALID_ARG;
    const d2d_layer_desc &D = layer->desc;
    int p = layer->expert_path;
    if (p == D2D_PATH_FUSED && layer->fused_group <= 0) return D2D_ERR_UNSUPPORTED;
    if (p != D2D_PATH_FUSED && layer->gather_group <= 0) p = D2D_PATH_DENSE;
    if (p == D2D_PATH_AUTO) {
        const double up_flop = 2.0 * (double)T * D.d * D.d_ff * (D.gated ? 2.0 : 1.0);
        const double pairs = (double)T * (double)D.n_experts;
        const double rho_max = layer->gather_rho_max >= 0.0 ? layer->gather_rho_max : default_gather_rho_max(D, layer->gather_group, T);
        if (up_flop < kAutoMinUpFlop) p = D2D_PATH_DENSE;
        else if (layer->fused_group > 0 && layer->fused_rho_max > 0.0 && n_sel <= (long long)(layer->fused_rho_max * pairs)) p = D2D_PATH_FUSED;
        else if (n_sel <= (long long)(rho_max * pairs) || (layer->fused_group > 0 && n_sel <= (long long)(layer->fused_rho_max * pairs))) p = D2D_PATH_GATHER;
        else p = D2D_PATH_DENSE;
    }
    *path = p;
    return D2D_OK;
}

d2d_status d2d_layer_get_fused(const d2d_layer *layer, int32_t *group, double *rho_max)
{
    if (!layer) return D2D_ERR_INVALID_ARG;
    if (group) *group = layer->fused_group;
    if (rho_max) *rho_max = layer->fused_rho_max;
    return D2D_OK;
}

d2d_status d2d_layer_get_expert_path(const d2d_layer *layer, int32_t *path, int32_t *group, double *rho_max)
{
    if (!layer) return D2D_ERR_INVALID_ARG;
    if (path) *path = layer->expert_path;
    if (group) *group = layer->expert_path == D2D_PATH_FUSED ? layer->fused_group : layer->gather_group;
    if (rho_max) *rho_max = layer->gather_rho_max;
    return D2D_OK;
}

d2d_status d2d_layer_reset_counters(d2d_layer *layer, void *stream)
{
    if (!layer) return D2D_ERR_INVALID_ARG;
    const size_t bytes = 256 + d2d_align_up((size_t)layer->gather_ctr_words * sizeof(int), 256);
    return cudaMemsetAsync(layer->slab, 0, bytes, (cudaStream_t)stream) == cudaSuccess ? D2D_OK : D2D_ERR_CUDA;
}

size_t d2d_workspace_bytes(const d2d_layer *layer, int32_t max_tokens)
{
    if (!layer || max_tokens < 0) return 0;
    return layout_for(layer, max_tokens).total;
}

size_t d2d_select_workspace_bytes(int32_t T, int32_t E)
{
    if (T < 0 || E <= 0) return 0;
    return d2d_select_ws_bytes(T, E);
}

d2d_status d2d_router_fwd(const d2d_layer *layer, const void *x, int32_t T, float *R,
                          void *ws, size_t ws_bytes, void *stream)
{
    if (!layer || T < 0) return D2D_ERR_INVALID_ARG;
    if (T == 0) return D2D_OK;
    if (!x || !R || !ws || !aligned16(x) || !aligned16(R) || !aligned16(ws)) return D2D_ERR_INVALID_ARG;
    const ws_layout w = layout_for(layer, T);
    if (ws_bytes < w.total) return D2D_ERR_WORKSPACE;
    return d2d_launch_router(layer, x, T, R, (float *)((char *)ws + w.u_off), (cudaStream_t)stream);
}

static d2d_status select_common(const float *R, int32_t T, int32_t E, float tau, int topk, d2d_routing *out,
                                void *ws, size_t ws_bytes, void *stream, bool mask_is_input)
{
    if (T < 0 || E <= 0 || !routing_ok(out, false)) return D2D_ERR_INVALID_ARG;
    if (!mask_is_input && T > 0 && (!R || !aligned16(R))) return D2D_ERR_INVALID_ARG;
    if (!mask_is_input && topk == 0 && !(tau >= 0.0f && tau <= 1.0f)) return D2D_ERR_INVALID_ARG;   // also rejects NaN
    if (topk < 0 || (topk > 0 && E > 2048)) return topk < 0 ? D2D_ERR_INVALID_ARG : D2D_ERR_UNSUPPORTED;
    if (T > 0 && (!ws || ws_bytes < d2d_select_ws_bytes(T, E))) return D2D_ERR_WORKSPACE;
    return d2d_launch_select(mask_is_input ? nullptr : R, T, E, tau, topk, out, ws, (cudaStream_t)stream);
}

d2d_status d2d_select_dynk(const float *R, int32_t T, int32_t E, float tau, d2d_routing *out,
                           void *ws, size_t ws_bytes, void *stream)
{
    return select_common(R, T, E, tau, 0, out, ws, ws_bytes, stream, false);
}

d2d_status d2d_select_topk(const float *R, int32_t T, int32_t E, int32_t kk, d2d_routing *out,
                           void *ws, size_t ws_bytes, void *stream)
{
    if (kk <= 0) return D2D_ERR_INVALID_ARG;
    return select_common(R, T, E, 0.0f, kk, out, ws, ws_bytes, stream, false);
}

d2d_status d2d_routing_from_mask(int32_t T, int32_t E, d2d_routing *out, void *ws, size_t ws_bytes, void *stream)
{
    return select_common(nullptr, T, E, 0.0f, 0, out, ws, ws_bytes, stream, true);
}

d2d_status d2d_moe_ffn_fwd(const d2d_layer *layer, const void *x, int32_t T, const d2d_routing *routing,
                           void *y, void *ws, size_t ws_bytes, void *stream)
{
    if (!layer || T < 0) return D2D_ERR_INVALID_ARG;
    if (T == 0) return D2D_OK;
    if (!x || !y || !aligned16(x) || !aligned16(y) || !routing_ok(routing, false)) return D2D_ERR_INVALID_ARG;
    const ws_layout w = layout_for(layer, T);
    if (!ws || ws_bytes < w.total) return D2D_ERR_WORKSPACE;
    return d2d_launch_moe_ffn(layer, x, T, routing, y, (char *)ws + w.ffn_off, w.total - w.ffn_off,
                              (cudaStream_t)stream);
}

d2d_status d2d_expert_up_fwd(const d2d_layer *layer, const void *x, int32_t T, const d2d_routing *routing,
                             void *H, void *stream)
{
    if (!layer || T < 0) return D2D_ERR_INVALID_ARG;
    if (T == 0) return D2D_OK;
    if (!x || !H || !aligned16(x) || !aligned16(H) || !routing_ok(routing, false)) return D2D_ERR_INVALID_ARG;
    if (layer->desc.dtype != D2D_BF16 || layer->desc.d_ff % 8 || !d2d_gemm_tc_available()) return D2D_ERR_UNSUPPORTED;
    const d2d_layer_desc &D = layer->desc;
    d2d_gemm_args up = {};
    up.a = x; up.b = layer->w1; up.b_gate = D.gated ? layer->w_gate : nullptr; up.b_cat = layer->w1g; up.b_cat_block = 128; up.bias = layer->b1; up.out = H;
    up.M = T; up.N = D.d_ff; up.K = D.d; up.epilogue = D2D_EPI_UP_MASKED; up.act = D.act;
    up.mask = routing->mask; up.mask_words = (D.n_experts + 31) / 32; up.expert_size = D.expert_size;
    up.status = routing->status;
    up.test_skip_load = __atomic_exchange_n(&g_test_fault, 0, __ATOMIC_RELAXED) == 1;
    return d2d_gemm_tc(up, (cudaStream_t)stream);
}

d2d_status d2d_test_inject_fault(int32_t kind)
{
    if (kind != 0 && kind != 1) return D2D_ERR_INVALID_ARG;
    __atomic_store_n(&g_test_fault, kind, __ATOMIC_RELAXED);
    return D2D_OK;
}

d2d_status d2d_expert_up_gather_fwd(const d2d_layer *layer, const void *x, int32_t T, const d2d_routing *routing,
                                    void *H, void *stream)
{
    if (!layer || T < 0) return D2D_ERR_INVALID_ARG;
    if (T == 0) return D2D_OK;
    if (!x || !H || !aligned16(x) || !aligned16(H) || !routing_ok(routing, false)) return D2D_ERR_INVALID_ARG;
    if (layer->gather_group <= 0) return D2D_ERR_UNSUPPORTED;
    const d2d_layer_desc &D = layer->desc;
    d2d_gather_args ga = {};
    ga.x = x; ga.w1 = layer->w1; ga.w_gate = D.gated ? layer->w_gate : nullptr; ga.b1 = layer->b1; ga.mask = routing->mask; ga.H = H;
    ga.T = T; ga.d = D.d; ga.d_ff = D.d_ff; ga.n_experts = D.n_experts; ga.s = D.expert_size; ga.g = layer->gather_group;
    ga.act = D.act; ga.status = routing->status; ga.ctr = layer->gather_ctr;
    ga.n_sel = routing->n_sel; ga.n_sel_min = -1; ga.n_sel_max = LLONG_MAX;
    return d2d_moe_gather_up(ga, (cudaStream_t)stream);
}

d2d_status d2d_expert_down_masked_fwd(const d2d_layer *layer, const void *H, int32_t T, const d2d_routing *routing, void *y,
                                      void *stream)
{
    if (!layer || T < 0) return D2D_ERR_INVALID_ARG;
    if (T == 0) return D2D_OK;
    if (!H || !y || !aligned16(H) || !aligned16(y) || !routing_ok(routing, true)) return D2D_ERR_INVALID_ARG;
    if (!d2d_moe_down_masked_supports(layer->desc)) return D2D_ERR_UNSUPPORTED;
    return d2d_moe_down_masked(layer->desc, H, routing->mask, layer->w2, layer->b2, y, T, routing->status, (cudaStream_t)stream);
}

d2d_status d2d_expert_down_fwd(const d2d_layer *layer, const void *H, int32_t T, void *y, int32_t *status, void *stream)
{
    if (!layer || T < 0) return D2D_ERR_INVALID_ARG;
    if (T == 0) return D2D_OK;
    if (!H || !y || !aligned16(H) || !aligned16(y)) return D2D_ERR_INVALID_ARG;
    if (layer->desc.dtype != D2D_BF16 || layer->desc.d_ff % 8 || !d2d_gemm_tc_available()) return D2D_ERR_UNSUPPORTED;
    const d2d_layer_desc &D = layer->desc;
    d2d_gemm_args dn = {};
    dn.a = H; dn.b = layer->w2; dn.bias = layer->b2; dn.out = y;
    dn.M = T; dn.N = D.d; dn.K = D.d_ff; dn.epilogue = D2D_EPI_BIAS_BF16; dn.status = status;
    return d2d_gemm_tc(dn, (cudaStream_t)stream);
}

d2d_status d2d_layer_fwd(const d2d_layer *layer, const void *x, int32_t T, float tau, void *y,
                         float *R_out, d2d_routing *routing, void *ws, size_t ws_bytes, void *stream)
{
    if (!layer || T < 0 || !routing_ok(routing, true)) return D2D_ERR_INVALID_ARG;
    if (!(tau >= 0.0f && tau <= 1.0f)) return D2D_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const int E = layer->desc.n_experts;
    const bool lists = has_lists(routing);
    if (T == 0) return lists ? d2d_launch_select(nullptr, 0, E, tau, 0, routing, ws, st) : D2D_OK;
    if (!x || !y || !aligned16(x) || !aligned16(y) || (R_out && !aligned16(R_out))) return D2D_ERR_INVALID_ARG;
    const ws_layout w = layout_for(layer, T);
    if (!ws || !aligned16(ws) || ws_bytes < w.total) return D2D_ERR_WORKSPACE;
    char *base = (char *)ws;
    float *R = R_out ? R_out : (float *)(base + w.r_off);
    d2d_status rc;
    if (d2d_router_fused_supports(layer->desc, T)) {
        // router and dynamic-k mask in one kernel; the selection step then only builds the per-expert metadata
        if (cudaMemsetAsync(routing->status, 0, sizeof(int32_t), st) != cudaSuccess) return D2D_ERR_CUDA;
        const bool dense = use_dense_masked(layer, T) && !use_small_ffn(layer, T);
        // tile counter of the up projection: layer-owned, zero at creation and reset by the kernel that used it, so no
        // memset node sits in front of the router (the up projection may begin while the router is still running)
        int *up_counter = dense ? (int *)(layer->tickets + 32) : nullptr;
        // the scores themselves are written only when the caller asked for them: mask and k come out of the same kernel
        // the router also adds up k: the number of selected pairs, which decides between the two up projections
        int32_t *ksum = (int32_t *)(layer->tickets + 40);
        rc = d2d_router_fused(layer, x, T, tau, 1, R_out, routing->mask, routing->k, routing->status, st, dense ? ksum : nullptr);
        if (rc != D2D_OK) return rc;
        if (dense) {
            // The tensor-core expert kernels read only the mask: the per-expert lists (when the caller wants them) are
            // built on the side stream while they run (the small metadata CTAs fit beside the persistent CTAs), join at the end.
            if (lists) {
                if (cudaEventRecord(layer->ev_fork, st) != cudaSuccess ||
                    cudaStreamWaitEvent(layer->side_stream, layer->ev_fork, 0) != cudaSuccess)
                    return D2D_ERR_CUDA;
                rc = d2d_launch_select(nullptr, T, E, tau, 0, routing, base + w.sel_off, layer->side_stream, 1);
                if (rc != D2D_OK) return rc;
            }
            rc = d2d_launch_moe_ffn(layer, x, T, routing, y, base + w.ffn_off, w.total - w.ffn_off, st, up_counter, 0, ksum + 4);
            if (lists && (cudaEventRecord(layer->ev_join, layer->side_stream) != cudaSuccess ||
                          cudaStreamWaitEvent(st, layer->ev_join, 0) != cudaSuccess))
                return D2D_ERR_CUDA;
            return rc;
        }
        if (!lists) return D2D_ERR_INVALID_ARG;               // the expert kernels of this shape walk the per-expert lists
        rc = d2d_launch_select(nullptr, T, E, tau, 0, routing, base + w.sel_off, st, 1);
    } else if (T > 8 && d2d_layer_token_fused_supports(layer->desc, T, lists)) {
        // small float32 problems: router, rule, experts and lists in one launch
        if (cudaMemsetAsync(routing->status, 0, sizeof(int32_t), st) != cudaSuccess) return D2D_ERR_CUDA;
        return d2d_layer_token_fused(layer, x, T, tau, y, R_out, routing, lists, layer->tickets + 52, st);
    } else if (lists && d2d_small_router_supports(layer->desc, T)) {
        // decode batches: the router kernel's last CTA selects as well (one launch for router + selection)
        const bool small = use_small_ffn(layer, T);
        float *y32 = (float *)(base + w.ffn_off + 256);
        rc = d2d_small_router(layer, x, T, R, base + w.u_off, st, routing, tau, 1, small ? y32 : nullptr,
                              small ? T * layer->desc.d : 0);
        if (rc != D2D_OK) return rc;
        return d2d_launch_moe_ffn(layer, x, T, routing, y, base + w.ffn_off, w.total - w.ffn_off, st, nullptr, small ? 1 : 0);
    } else if (use_dense_masked(layer, T) && !use_small_ffn(layer, T) && !d2d_small_select_supports(T, E)) {
        // router shapes the fused kernel does not take, tensor-core expert step: scores by two GEMMs, then mask, k and
        // the number of selected pairs by one kernel; the per-expert lists (when wanted) are built on the side stream
        // while the experts, which read only the mask, run
        rc = d2d_launch_router(layer, x, T, R, (float *)(base + w.u_off), st);
        if (rc != D2D_OK) return rc;
        int32_t *ksum = (int32_t *)(layer->tickets + 40);
        rc = d2d_launch_dynk_mask(R, T, E, tau, routing, ksum, st);
        if (rc != D2D_OK) return rc;
        if (lists) {
            if (cudaEventRecord(layer->ev_fork, st) != cudaSuccess || cudaStreamWaitEvent(layer->side_stream, layer->ev_fork, 0) != cudaSuccess)
                return D2D_ERR_CUDA;
            rc = d2d_launch_select(nullptr, T, E, tau, 0, routing, base + w.sel_off, layer->side_stream, 1);
            if (rc != D2D_OK) return rc;
        }
        rc = d2d_launch_moe_ffn(layer, x, T, routing, y, base + w.ffn_off, w.total - w.ffn_off, st, nullptr, 0, ksum + 4);
        if (lists && (cudaEventRecord(layer->ev_join, layer->side_stream) != cudaSuccess || cudaStreamWaitEvent(st, layer->ev_join, 0) != cudaSuccess))
            return D2D_ERR_CUDA;
        return rc;
    } else if (!lists) {
        return D2D_ERR_INVALID_ARG;                           // every other path builds (and its expert kernels use) the lists
    } else {
        rc = d2d_launch_router(layer, x, T, R, (float *)(base + w.u_off), st);
        if (rc != D2D_OK) return rc;
        rc = d2d_launch_select(R, T, E, tau, 0, routing, base + w.sel_off, st);
    }
    if (rc != D2D_OK) return rc;
    return d2d_launch_moe_ffn(layer, x, T, routing, y, base + w.ffn_off, w.total - w.ffn_off, st);
}

// Data-dependent conditions of a finished host call: the largest device status word (0 = ok).
static d2d_status host_status(const int32_t *status_dev, int n)
{
    int32_t h[d2d_layer::kHostChunks] = {0, 0, 0, 0};
    if (n > d2d_layer::kHostChunks) n = d2d_layer::kHostChunks;
    if (cudaMemcpy(h, status_dev, sizeof(int32_t) * (size_t)n, cudaMemcpyDeviceToHost) != cudaSuccess) return D2D_ERR_CUDA;
    int32_t worst = 0;
    for (int i = 0; i < n; ++i) worst = h[i] > worst ? h[i] : worst;
    return (d2d_status)worst;
}

// Carves routing buffers + x/y staging + the layer workspace out of one device buffer.
struct host_call_layout {
    size_t x_off, y_off, mask_off, k_off, counts_off, offsets_off, perm_off, scalars_off, ws_off, total;
};

static host_call_layout host_layout(const d2d_layer *L, int T)
{
    host_call_layout h;
    const size_t Tn = (size_t)(T > 0 ? T : 1), E = (size_t)L->desc.n_experts, W = (E + 31) / 32;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off += d2d_align_up(bytes, 256); return o; };
    h.x_off = take(Tn * L->desc.d * L->elem);
    h.y_off = take(Tn * L->desc.d * L->elem);
    h.mask_off = take(Tn * W * 4);
    h.k_off = take(Tn * 4);
    h.counts_off = take(E * 4);
    h.offsets_off = take((E + 1) * 4);
    h.perm_off = take(Tn * E * 4);
    h.scalars_off = take((2 + d2d_layer::kHostChunks) * 4);     // n_sel, then one status word per chunk
    h.ws_off = off;
    off += layout_for(L, (int)Tn).total;
    h.total = off;
    return h;
}

size_t d2d_layer_fwd_host_workspace_bytes(const d2d_layer *layer, int32_t max_tokens)
{
    if (!layer || max_tokens < 0) return 0;
    return host_layout(layer, max_tokens).total;
}

d2d_status d2d_layer_fwd_host(const d2d_layer *layer, const void *x_host, int32_t T, float tau, void *y_host,
                              void *ws, size_t ws_bytes, void *stream)
{
    if (!layer || T < 0) return D2D_ERR_INVALID_ARG;
    if (T == 0) return D2D_OK;
    if (!x_host || !y_host || !ws || !aligned16(ws)) return D2D_ERR_INVALID_ARG;
    const host_call_layout h = host_layout(layer, T);
    if (ws_bytes < h.total) return D2D_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    char *base = (char *)ws;
    const size_t tok_bytes = (size_t)layer->desc.d * layer->elem;
    const size_t row_bytes = (size_t)T * tok_bytes;
    d2d_routing r;
    memset(&r, 0, sizeof(r));
    r.mask = (uint32_t *)(base + h.mask_off);
    r.k = (int32_t *)(base + h.k_off);
    r.counts = (int32_t *)(base + h.counts_off);
    r.offsets = (int32_t *)(base + h.offsets_off);
    r.perm = (int32_t *)(base + h.perm_off);
    r.n_sel = (int32_t *)(base + h.scalars_off);
    r.status = r.n_sel + 1;
    r.perm_capacity = (int64_t)T * layer->desc.n_experts;
    // Tokens are independent, so a large batch is cut into chunks (multiples of 128 tokens) and pipelined: the copy of
    // chunk c+1 to the device (copy-in stream), the layer on chunk c (`stream`) and the copy of chunk c-1 back to the
    // host (copy-out stream) run at the same time; PCIe carries both directions at once.  The routing buffers and the
    // layer workspace are reused chunk after chunk, which is safe because the layer calls are serial on `stream`.
    // The layer is the slowest of the three legs for the shapes where this matters, so the whole call takes about
    // (copy-in of the first chunk) + (all layer calls) + (copy-out of the last chunk): the first and the last chunk
    // are short, the ones in between long (a short chunk costs more per token, so there are few of them).
    int bounds[d2d_layer::kHostChunks + 1] = {0, T, T, T, T};
    int n_chunks = 1;
    if (T >= 8192) {
        // sizes 3T/16, 5T/16, 5T/16, 3T/16 in multiples of 128 tokens (measured on the Llama-shaped layer, 8192 tokens:
        // 2.50 ms; T/8, 3T/8, 3T/8, T/8: 2.64; four equal chunks: 2.62; two equal chunks: 3.04)
        const int a = d2d_cdiv(3 * (T / 16), 128) * 128, b = d2d_cdiv((T - 2 * a) / 2, 128) * 128;
        bounds[1] = a; bounds[2] = a + b; bounds[3] = T - a > a + b ? T - a : a + b; bounds[4] = T;
        n_chunks = 4;
    }
    if (const char *e = getenv("D2D_HOST_CHUNKS")) {          // 1 .. 4 equal chunks, for tuning
        const int n = atoi(e);
        if (n >= 1 && n <= d2d_layer::kHostChunks && T >= 128 * n) {
            n_chunks = n;
            const int chunk = d2d_cdiv(d2d_cdiv(T, n), 128) * 128;
            for (int c = 1; c <= d2d_layer::kHostChunks; ++c) bounds[c] = c * chunk < T && c < n ? c * chunk : T;
        }
    }
    if (n_chunks == 1) {
        D2D_CUDA_TRY(cudaMemcpyAsync(base + h.x_off, x_host, row_bytes, cudaMemcpyHostToDevice, st));
        d2d_status rc = d2d_layer_fwd(layer, base + h.x_off, T, tau, base + h.y_off, nullptr, &r,
                                      base + h.ws_off, h.total - h.ws_off, st);
        if (rc != D2D_OK) return rc;
        D2D_CUDA_TRY(cudaMemcpyAsync(y_host, base + h.y_off, row_bytes, cudaMemcpyDeviceToHost, st));
        D2D_CUDA_TRY(cudaStreamSynchronize(st));
        return host_status(r.status, 1);
    }
    // the copies may not start before work already queued on `stream` (which may still use ws) has finished
    D2D_CUDA_TRY(cudaEventRecord(layer->ev_begin, st));
    D2D_CUDA_TRY(cudaStreamWaitEvent(layer->copy_in, layer->ev_begin, 0));
    D2D_CUDA_TRY(cudaStreamWaitEvent(layer->copy_out, layer->ev_begin, 0));
    for (int c = 0; c < n_chunks; ++c) {
        const int t0 = bounds[c], tc = bounds[c + 1] - bounds[c];
        if (tc <= 0) continue;
        D2D_CUDA_TRY(cudaMemcpyAsync(base + h.x_off + (size_t)t0 * tok_bytes, (const char *)x_host + (size_t)t0 * tok_bytes,
                                     (size_t)tc * tok_bytes, cudaMemcpyHostToDevice, layer->copy_in));
        D2D_CUDA_TRY(cudaEventRecord(layer->ev_in[c], layer->copy_in));
    }
    d2d_status rc = D2D_OK;
    int32_t *const status0 = r.status;
    int n_used = 0;
    for (int c = 0; c < n_chunks; ++c) {
        const int t0 = bounds[c], tc = bounds[c + 1] - bounds[c];
        if (tc <= 0) continue;
        r.status = status0 + n_used;                         // one status word per chunk (the layer call clears its own)
        ++n_used;
        D2D_CUDA_TRY(cudaStreamWaitEvent(st, layer->ev_in[c], 0));
        rc = d2d_layer_fwd(layer, base + h.x_off + (size_t)t0 * tok_bytes, tc, tau, base + h.y_off + (size_t)t0 * tok_bytes,
                           nullptr, &r, base + h.ws_off, h.total - h.ws_off, st);
        if (rc != D2D_OK) break;
        D2D_CUDA_TRY(cudaEventRecord(layer->ev_done[c], st));
        D2D_CUDA_TRY(cudaStreamWaitEvent(layer->copy_out, layer->ev_done[c], 0));
        D2D_CUDA_TRY(cudaMemcpyAsync((char *)y_host + (size_t)t0 * tok_bytes, base + h.y_off + (size_t)t0 * tok_bytes,
                                     (size_t)tc * tok_bytes, cudaMemcpyDeviceToHost, layer->copy_out));
    }
    // join both copy streams back into `stream` (also on the error path, so nothing is left running on them)
    cudaEventRecord(layer->ev_end, layer->copy_out);
    cudaStreamWaitEvent(st, layer->ev_end, 0);
    cudaEventRecord(layer->ev_end, layer->copy_in);
    cudaStreamWaitEvent(st, layer->ev_end, 0);
    if (rc != D2D_OK) return rc;
    D2D_CUDA_TRY(cudaStreamSynchronize(st));
    return host_status(status0, n_used);
}

}  // extern "C"
