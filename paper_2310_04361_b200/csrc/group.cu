// Layer groups: several dynamic-k layers of one shape that read the same token rows, run as one launch sequence.
// In a converted Transformer block the Q, K and V projections of the attention layer are such a group (Sec. 3.5: every
// projection matrix becomes its own MoE layer, four of them per attention layer); the output projection and the FFN
// read other tensors and stay ordinary d2d_layer_fwd calls.
//
//   T <= decode limit   one decode router launch (+ selection + metadata) and one expert launch for all layers
//                       (grid.y = layer), instead of two launches per layer
//   larger bf16 batches the routers run as one tcgen05 grid (grid.y = layer) that also writes a merged selection mask
//                       [T, n*ceil(E/32)]; the up projections are ONE GEMM over the stacked W1 ([n*d_ff, d]: the token
//                       tile is read once for all layers, 3x the tiles to balance over the SMs); the down projections
//                       are one batched GEMM (problem l reads column block l of the merged hidden activations)
//   anything else       the layers run one after the other through d2d_layer_fwd
#include <new>
#include <string.h>

#include "d2d_common.cuh"
#include "gemm_tc.cuh"

namespace {

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool same_shape(const d2d_layer_desc &a, const d2d_layer_desc &b)
{
    return a.d == b.d && a.d_ff == b.d_ff && a.n_experts == b.n_experts && a.expert_size == b.expert_size && a.d_h == b.d_h &&
           a.dtype == b.dtype && a.act == b.act && a.gated == b.gated;
}

bool routing_full(const d2d_routing *r)
{
    if (!r->mask || !r->k || !r->counts || !r->offsets || !r->perm || !r->n_sel || !r->status) return false;
    if ((r->tok_off == nullptr) != (r->tok_exp == nullptr)) return false;
    return r->perm_capacity >= 0;
}

// Workspace of d2d_group_fwd.
struct group_layout {
    size_t sel_off, sel_each;      // per-layer selection scratch
    size_t r_off, r_each;          // per-layer scores (decode path)
    size_t u_off, u_each;          // per-layer router hidden activations (decode path)
    size_t y32_off, y32_each;      // per-layer float32 output accumulators (decode path)
    size_t mask_off;               // merged mask [T, n*W]
    size_t h_off;                  // merged hidden activations [T, n*d_ff] bf16
    size_t partial_off;            // split-K sums of the batched down projection [n, T, d] float32
    size_t seq_off;                // workspace of the sequential fallback
    size_t total;
};

group_layout layout_for(const d2d_group *g, int T)
{
    const d2d_layer_desc &D = g->desc;
    const size_t Tn = (size_t)(T > 0 ? T : 1), n = (size_t)g->n;
    const size_t W = (size_t)(D.n_experts + 31) / 32;
    group_layout w;
    size_t off = 0;
    w.sel_off = off; w.sel_each = d2d_align_up(d2d_select_ws_bytes((int)Tn, D.n_experts), 256); off += n * w.sel_each;
    const bool decode = (int)Tn <= 8;
    w.r_off = off; w.r_each = decode ? d2d_align_up(Tn * D.n_experts * 4, 256) : 0; off += n * w.r_each;
    w.u_off = off; w.u_each = decode ? d2d_align_up(Tn * D.d_h * 4, 256) : 0; off += n * w.u_each;
    w.y32_off = off; w.y32_each = decode ? d2d_align_up(Tn * D.d * 4, 256) : 0; off += n * w.y32_each;
    w.mask_off = off;
    if (g->merged) off += d2d_align_up(Tn * n * W * 4, 256);
    w.h_off = off;
    if (g->merged) off += d2d_align_up(Tn * n * D.d_ff * 2, 256);
    w.partial_off = off;
    if (g->merged && d2d_gemm_tc_splits((int)Tn, D.d, D.d_ff, g->n) > 1) off += d2d_align_up(n * Tn * D.d * 4, 256);
    w.seq_off = off;
    off += d2d_workspace_bytes(g->layers[0], (int)Tn);
    w.total = off;
    return w;
}

}  // namespace

extern "C" {

d2d_status d2d_group_create(d2d_layer *const *layers, int32_t n_layers, void *stream, d2d_group **out)
{
    if (out) *out = nullptr;
    if (!layers || !out || n_layers < 1 || n_layers > D2D_MAX_GROUP) return D2D_ERR_INVALID_ARG;
    for (int l = 0; l < n_layers; ++l) {
        if (!layers[l] || !same_shape(layers[l]->desc, layers[0]->desc)) return D2D_ERR_INVALID_ARG;
        for (int m = 0; m < l; ++m)
            if (layers[m] == layers[l]) return D2D_ERR_INVALID_ARG;     // a layer's tickets serve one grid row
    }
    d2d_group *g = new (std::nothrow) d2d_group();
    if (!g) return D2D_ERR_CUDA;
    memset(g, 0, sizeof(*g));
    g->n = n_layers;
    for (int l = 0; l < n_layers; ++l) g->layers[l] = layers[l];
    const d2d_layer_desc &D = layers[0]->desc;
    g->desc = D;
    // the merged tensor-core path: bf16, plain (not gated) experts, the fused router's shape, and whole mask words per
    // layer so that expert e of layer l is bit l*E + e of the merged mask
    g->merged = D.dtype == D2D_BF16 && !D.gated && D.d_h == 128 && D.n_experts <= 256 && D.n_experts % 32 == 0 &&
                D.d_ff % 64 == 0 && D.d % 8 == 0 && d2d_gemm_tc_available();
    cudaStream_t st = (cudaStream_t)stream;
    d2d_status rc = D2D_OK;
    if (g->merged) {
        const size_t el = 2, n = (size_t)n_layers;
        struct piece { void **dst; size_t each; size_t off_in_layer; } pieces[] = {
            {&g->w_r1, (size_t)D.d_h * D.d * el, offsetof(d2d_layer, w_r1)}, {&g->b_r1, (size_t)D.d_h * el, offsetof(d2d_layer, b_r1)},
            {&g->w_r2, (size_t)D.n_experts * D.d_h * el, offsetof(d2d_layer, w_r2)}, {&g->b_r2, (size_t)D.n_experts * el, offsetof(d2d_layer, b_r2)},
            {&g->w1, (size_t)D.d_ff * D.d * el, offsetof(d2d_layer, w1)}, {&g->b1, (size_t)D.d_ff * el, offsetof(d2d_layer, b1)},
            {&g->w2, (size_t)D.d * D.d_ff * el, offsetof(d2d_layer, w2)}, {&g->b2, (size_t)D.d * el, offsetof(d2d_layer, b2)},
        };
        size_t total = 256;
        for (const piece &p : pieces) total += d2d_align_up(n * p.each, 256);
        if (cudaMalloc(&g->slab, total) != cudaSuccess) {
            delete g;
            return D2D_ERR_CUDA;
        }
        // zero: the tile counter, and the entries of a bias some layer does not have
        if (cudaMemsetAsync(g->slab, 0, total, st) != cudaSuccess) rc = D2D_ERR_CUDA;
        g->up_counter = (int *)g->slab;
        size_t off = 256;
        for (const piece &p : pieces) {
            char *dst = (char *)g->slab + off;
            off += d2d_align_up(n * p.each, 256);
            *p.dst = dst;
            for (int l = 0; l < n_layers && rc == D2D_OK; ++l) {
                const void *src = *(void *const *)((const char *)layers[l] + p.off_in_layer);
                if (src && cudaMemcpyAsync(dst + (size_t)l * p.each, src, p.each, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
                    rc = D2D_ERR_CUDA;
            }
        }
        if (rc == D2D_OK && cudaStreamSynchronize(st) != cudaSuccess) rc = D2D_ERR_CUDA;
    }
    if (rc == D2D_OK && (cudaStreamCreateWithFlags(&g->side_stream, cudaStreamNonBlocking) != cudaSuccess ||
                         cudaEventCreateWithFlags(&g->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
                         cudaEventCreateWithFlags(&g->ev_join, cudaEventDisableTiming) != cudaSuccess))
        rc = D2D_ERR_CUDA;
    if (rc != D2D_OK) {
        d2d_group_destroy(g);
        return rc;
    }
    *out = g;
    return D2D_OK;
}

d2d_status d2d_group_destroy(d2d_group *g)
{
    if (!g) return D2D_OK;
    if (g->ev_join) cudaEventDestroy(g->ev_join);
    if (g->ev_fork) cudaEventDestroy(g->ev_fork);
    if (g->side_stream) cudaStreamDestroy(g->side_stream);
    const cudaError_t e = g->slab ? cudaFree(g->slab) : cudaSuccess;
    delete g;
    return e == cudaSuccess ? D2D_OK : D2D_ERR_CUDA;
}

size_t d2d_group_workspace_bytes(const d2d_group *g, int32_t max_tokens)
{
    if (!g || max_tokens < 0) return 0;
    return layout_for(g, max_tokens).total;
}

d2d_status d2d_group_fwd(const d2d_group *g, const void *x, int32_t T, float tau, void *y, d2d_routing *routing,
                         void *ws, size_t ws_bytes, void *stream)
{
    if (!g || T < 0 || !routing) return D2D_ERR_INVALID_ARG;
    if (!(tau >= 0.0f && tau <= 1.0f)) return D2D_ERR_INVALID_ARG;
    for (int l = 0; l < g->n; ++l)
        if (!routing_full(&routing[l])) return D2D_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const d2d_layer_desc &D = g->desc;
    const int n = g->n, E = D.n_experts;
    const size_t el = g->layers[0]->elem;
    if (T == 0) {
        for (int l = 0; l < n; ++l) {
            const d2d_status rc = d2d_launch_select(nullptr, 0, E, tau, 0, &routing[l], ws, st);
            if (rc != D2D_OK) return rc;
        }
        return D2D_OK;
    }
    if (!x || !y || !aligned16(x) || !aligned16(y) || ((size_t)T * D.d * el) % 16) return D2D_ERR_INVALID_ARG;
    const group_layout w = layout_for(g, T);
    if (!ws || !aligned16(ws) || ws_bytes < w.total) return D2D_ERR_WORKSPACE;
    char *base = (char *)ws;

    // ---- decode batches: two launches for the whole group
    if (d2d_small_router_supports(D, T) && d2d_small_ffn_supports(D) && T <= (D.dtype == D2D_BF16 ? d2d_decode_max_tokens(D) : 8)) {
        float *R[D2D_MAX_GROUP], *u[D2D_MAX_GROUP], *y32[D2D_MAX_GROUP];
        for (int l = 0; l < n; ++l) {
            R[l] = (float *)(base + w.r_off + (size_t)l * w.r_each);
            u[l] = (float *)(base + w.u_off + (size_t)l * w.u_each);
            y32[l] = (float *)(base + w.y32_off + (size_t)l * w.y32_each);
        }
        return d2d_small_group_fwd(g->layers, n, x, T, tau, routing, R, u, y32, y, st);
    }

    // ---- merged tensor-core path
    if (g->merged && d2d_router_fused_supports(D, T)) {
        const int W = E / 32;
        for (int l = 0; l < n; ++l)
            if (cudaMemsetAsync(routing[l].status, 0, sizeof(int32_t), st) != cudaSuccess) return D2D_ERR_CUDA;
        uint32_t *mask_cat = (uint32_t *)(base + w.mask_off);
        const d2d_router_weights rw = {g->w_r1, g->b_r1, g->w_r2, g->b_r2};
        d2d_status rc = d2d_router_fused_group(D, rw, n, x, T, tau, routing, mask_cat, n * W, st);
        if (rc != D2D_OK) return rc;
        // per-expert metadata of every layer on the side stream, beside the GEMMs (which read only the merged mask)
        if (cudaEventRecord(g->ev_fork, st) != cudaSuccess || cudaStreamWaitEvent(g->side_stream, g->ev_fork, 0) != cudaSuccess)
            return D2D_ERR_CUDA;
        for (int l = 0; l < n; ++l) {
            rc = d2d_launch_select(nullptr, T, E, tau, 0, &routing[l], base + w.sel_off + (size_t)l * w.sel_each, g->side_stream, 1);
            if (rc != D2D_OK) return rc;
        }
        void *H = base + w.h_off;
        d2d_gemm_args up = {};
        up.tile_counter = g->up_counter;
        up.pdl_late_wait = 1;                       // x and the weights do not depend on the router, only the mask does
        up.a = x; up.b = g->w1; up.bias = g->b1; up.out = H;
        up.M = T; up.N = n * D.d_ff; up.K = D.d; up.epilogue = D2D_EPI_UP_MASKED; up.act = D.act;
        up.mask = mask_cat; up.mask_words = n * W; up.expert_size = D.expert_size; up.status = routing[0].status;
        rc = d2d_gemm_tc(up, st);
        if (rc != D2D_OK) return rc;
        d2d_gemm_args dn = {};
        dn.a = H; dn.b = g->w2; dn.bias = g->b2; dn.out = y;
        dn.M = T; dn.N = D.d; dn.K = D.d_ff; dn.batch = n; dn.epilogue = D2D_EPI_BIAS_BF16; dn.status = routing[0].status;
        dn.k_splits = d2d_gemm_tc_splits(T, D.d, D.d_ff, n);
        dn.partial = dn.k_splits > 1 ? (float *)(base + w.partial_off) : nullptr;
        rc = d2d_gemm_tc(dn, st);
        if (cudaEventRecord(g->ev_join, g->side_stream) != cudaSuccess || cudaStreamWaitEvent(st, g->ev_join, 0) != cudaSuccess)
            return D2D_ERR_CUDA;
        return rc;
    }

    // ---- any other shape: one layer after the other
    for (int l = 0; l < n; ++l) {
        const d2d_status rc = d2d_layer_fwd(g->layers[l], x, T, tau, (char *)y + (size_t)l * T * D.d * el, nullptr, &routing[l],
                                            base + w.seq_off, w.total - w.seq_off, st);
        if (rc != D2D_OK) return rc;
    }
    return D2D_OK;
}

}  // extern "C"
