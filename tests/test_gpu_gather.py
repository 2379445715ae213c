"""GPU parity of the gathered, grouped expert path (tokens bucketed by groups of adjacent experts, Sec. 3.4 /
Listing 1) and of the density-adaptive dispatch between it and the masked dense up projection.

Every case runs the same inputs through each side of the dispatch (forced through d2d_layer_set_expert_path)
and through the automatic choice, and compares y with the CPU oracle on the same mask.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2310_04361_b200 import workloads as wl

pytestmark = pytest.mark.gpu

TOL_Y = 2e-2          # bf16 in/out, float32 accumulation: max|y - y_ref| / max|y_ref|


@pytest.fixture(scope="module")
def api():
    from paper_2310_04361_b200 import api as _api
    assert torch.cuda.is_available()
    return _api


def _rel_err(got, ref):
    ref = np.asarray(ref, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    return float(np.abs(got - ref).max() / max(np.abs(ref).max(), 1e-30))


def _per_token_err(got, ref):
    """max_t ( max_j |got - ref| / max_j |ref| ): every token normalised by its own magnitude."""
    ref = np.asarray(ref, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    return float((np.abs(got - ref).max(1) / np.maximum(np.abs(ref).max(1), 1e-30)).max())


def _config(name):
    """Workload by name; "wide" is a plain GELU layer with d = 2048 (the only plain shape here on which the gathered path
    zero-fills H and keeps the TMA-fed down projection, and on which all three ranges of the automatic choice exist)."""
    if name == "wide":
        import dataclasses
        return dataclasses.replace(wl.CONFIGS["bert"], name="wide", d=2048, d_ff=4096, T=12288, seed=9)
    return wl.CONFIGS[name]


def _routing(api, G, E):
    return api.routing_from_mask(torch.from_numpy(oracle.pack_mask(G).view(np.int32)).cuda(), E)


def _structured_mask(cfg, T, p, seed):
    """Bernoulli(p) with the degenerate columns and rows the bucketing has to survive: an expert nobody keeps, an
    expert everybody keeps, a token that keeps nothing, a token that keeps everything."""
    rng = np.random.default_rng(seed)
    G = (rng.random((T, cfg.E)) < p).astype(np.uint8)
    G[:, 1 % cfg.E] = 0
    G[:, (cfg.E - 2) % cfg.E] = 1
    G[T // 3] = 0
    G[T // 2] = 1
    return G


# (workload, tokens, experts per group or 0 = default, densities)
GATHER_CASES = [
    ("bert", 700, 0, (0.0, 0.03, 0.3, 1.0)),        # s = 24, default g = 4 (96 columns), ragged 256-token sub-chunk
    ("bert", 1024, 2, (0.2,)),                      # 48-column groups
    ("bert", 1300, 8, (0.1,)),                      # 192-column groups
    ("vit", 900, 0, (0.05, 0.5)),                   # s = 16, g = 8
    ("vit", 515, 4, (0.3,)),                        # 64-column groups
    ("paper", 2100, 0, (0.0, 0.3, 1.0)),            # s = 128, one expert per group (the paper's benchmark shape)
    ("llama", 600, 0, (0.1, 0.6)),                  # gated, s = 32, g = 4: one MMA fills the up and gate accumulators
    ("llama", 257, 2, (0.4,)),
    ("gpt2_ffn", 513, 0, (0.15,)),                  # d = 1024
]


@pytest.mark.parametrize("name,T,g,ps", GATHER_CASES)
def test_gathered_up_projection_equals_masked_dense_and_oracle(api, name, T, g, ps):
    cfg = wl.with_tokens(wl.CONFIGS[name], T)
    w, x = wl.make_weights(cfg), wl.make_tokens(cfg)
    layer = api.Layer.from_config(cfg, w)
    layer.set_expert_path("auto", group=g)
    xd = api.to_device(x, cfg.dtype)
    act = oracle.ACT_BY_NAME[cfg.act]
    for i, p in enumerate(ps):
        G = _structured_mask(cfg, T, p, seed=17 * i + T) if 0.0 < p < 1.0 else np.full((T, cfg.E), int(p), np.uint8)
        r = _routing(api, G, cfg.E)
        H_dense = layer.expert_up_fwd(xd, r).view(torch.int16).cpu().numpy().reshape(T, cfg.E, cfg.s)
        gg = layer.get_expert_path()[1]
        kept_group = np.repeat(G.reshape(T, cfg.E // gg, gg).max(-1), gg, axis=1).astype(bool)     # [T, E]: some expert of the group kept
        POISON = 0x7fc1                                        # a NaN pattern: cells the kernel must not touch, and must never read
        H = torch.full((T, cfg.d_ff), POISON, dtype=torch.int16, device="cuda").view(torch.bfloat16)
        y_ref = oracle.moe_ffn(x, w["w1"], w["b1"], w["w_gate"], w["w2"], w["b2"], act, G)
        for rep in range(2):                                   # twice: the sub-chunk counters reset themselves
            layer.expert_up_gather_fwd(xd, r, H=H)
            torch.cuda.synchronize()
            assert r.status == 0
            Hn = H.view(torch.int16).cpu().numpy().reshape(T, cfg.E, cfg.s)
            # cells of kept (token, group) pairs: bit for bit what the masked dense kernel writes (the same products
            # accumulated in the same order on the same unit), zero at experts of the group the token did not keep
            assert np.array_equal(Hn[kept_group], H_dense[kept_group]), (name, p)
            assert not Hn[kept_group & (G == 0)].any()
            # every other cell is left alone ...
            assert (Hn[~kept_group] == np.int16(POISON)).all()
            # ... and the down projection that follows never reads it
            y = layer.expert_down_masked_fwd(H, r).float().cpu().numpy()
            assert np.isfinite(y).all()
            assert _rel_err(y, y_ref) <= TOL_Y, (name, p, _rel_err(y, y_ref))
            H.view(torch.int16).fill_(POISON)
        # the same down projection after the masked dense kernel
        y = layer.expert_down_masked_fwd(layer.expert_up_fwd(xd, r), r).float().cpu().numpy()
        assert _rel_err(y, y_ref) <= TOL_Y
    layer.close()


PATH_CASES = [("bert", 1000, 0.5), ("bert", 640, 0.9), ("vit", 1500, 0.6), ("paper", 1500, 0.3), ("llama", 520, 0.6), ("wide", 700, 0.5)]


@pytest.mark.parametrize("name,T,tau", PATH_CASES)
def test_layer_fwd_is_the_same_on_both_sides_of_the_dispatch(api, name, T, tau):
    """d2d_layer_fwd and d2d_moe_ffn_fwd with the up projection forced dense, forced gathered, and chosen on the
    device with the crossover moved to either extreme: identical masks, y equal to the oracle's on that mask."""
    cfg = wl.with_tokens(_config(name), T)
    w, x = wl.make_weights(cfg), wl.make_tokens(cfg)
    layer = api.Layer.from_config(cfg, w)
    xd = api.to_device(x, cfg.dtype)
    act = oracle.ACT_BY_NAME[cfg.act]
    ref_mask, y_ref = None, None
    settings = [("dense", -1.0), ("gather", -1.0), ("auto", 0.0), ("auto", 1.0), ("auto", -1.0)]
    for path, rho_max in settings:
        layer.set_expert_path(path, rho_max=rho_max)
        for lists in (True, False):
            r = layer.new_routing(T, lists=lists)
            y = torch.full((T, cfg.d), float("nan"), dtype=torch.bfloat16, device="cuda")
            for rep in range(2):
                layer.layer_fwd(xd, tau, y=y, routing=r)
                torch.cuda.synchronize()
                assert r.status == 0
            m = r.mask_u32().copy()
            if ref_mask is None:
                ref_mask = m
                G = oracle.unpack_mask(m, cfg.E)
                y_ref = oracle.moe_ffn(x, w["w1"], w["b1"], w["w_gate"], w["w2"], w["b2"], act, G)
            assert np.array_equal(m, ref_mask)
            assert r.n_sel == int(oracle.unpack_mask(m, cfg.E).sum())
            yg = y.float().cpu().numpy()
            assert np.isfinite(yg).all()
            assert _rel_err(yg, y_ref) <= TOL_Y, (path, rho_max, lists, _rel_err(yg, y_ref))
            assert _per_token_err(yg, y_ref) <= 4 * TOL_Y, (path, rho_max, lists, _per_token_err(yg, y_ref))
        # the stand-alone expert step on the same mask
        r2 = _routing(api, oracle.unpack_mask(ref_mask, cfg.E), cfg.E)
        y2 = layer.moe_ffn_fwd(xd, r2).float().cpu().numpy()
        assert _rel_err(y2, y_ref) <= TOL_Y
    layer.close()


@pytest.mark.parametrize("name,tau", [("paper", 0.5), ("llama", 0.6), ("wide", 0.5)])
def test_device_side_choice_at_full_size(api, name, tau):
    """Batches large enough for the automatic choice: the crossover is moved to either extreme so that the decision
    taken on the device goes each way (both kernel pairs are enqueued, one returns at once); y is checked against
    the oracle on sampled tokens, at least one from every 128-token row tile."""
    cfg = _config(name)
    w, x = wl.make_weights(cfg), wl.make_tokens(cfg)
    layer = api.Layer.from_config(cfg, w)
    xd = api.to_device(x, cfg.dtype)
    act = oracle.ACT_BY_NAME[cfg.act]
    T = cfg.T
    rng = np.random.default_rng(11)
    tiles = np.arange(0, T, 128)
    sample = np.unique(np.concatenate([tiles + rng.integers(0, 128, tiles.shape), [0, T - 1]]))
    sample = sample[sample < T]
    if name in ("llama", "wide"):
        sample = sample[:: 2]                                  # the oracle needs about 0.1 s per Llama-sized token
    ref = None
    # (crossover of the gathered pair, upper end of the fused kernel's range): dense pair, gathered pair, fused kernel,
    # and the defaults
    settings = [(0.0, 0.0), (1.0, 0.0), (-1.0, -1.0)] + ([] if cfg.gated else [(0.0, 1.0)])
    for rho_max, fused_max in settings:
        layer.set_expert_path("auto", rho_max=rho_max)
        if not cfg.gated:
            layer.set_fused_rho_max(fused_max)
        r = layer.new_routing(T)
        y = torch.full((T, cfg.d), float("nan"), dtype=torch.bfloat16, device="cuda")
        for rep in range(2):
            layer.layer_fwd(xd, tau, y=y, routing=r)
            torch.cuda.synchronize()
            assert r.status == 0
        G = oracle.unpack_mask(r.mask_u32(), cfg.E)
        assert r.n_sel == int(G.sum())
        if (rho_max, fused_max) != (-1.0, -1.0):               # the host-side copy of the rule agrees with the setting
            want = "fused" if fused_max == 1.0 else "gather" if rho_max == 1.0 else "dense"
            assert layer.expert_path_for(T, r.n_sel) == want
        if ref is None:
            ref = (G, oracle.moe_ffn(x[sample], w["w1"], w["b1"], w["w_gate"], w["w2"], w["b2"], act, G[sample]))
        assert np.array_equal(G, ref[0])
        yg = y.float().cpu().numpy()
        assert np.isfinite(yg).all()
        assert _rel_err(yg[sample], ref[1]) <= TOL_Y, (rho_max, fused_max, _rel_err(yg[sample], ref[1]))
        assert _per_token_err(yg[sample], ref[1]) <= 4 * TOL_Y
    if cfg.gated:                                              # the fused kernel takes plain layers only
        with pytest.raises(api.D2DError) as e:
            layer.set_fused_rho_max(0.5)
        assert api.STATUS_NAMES[e.value.code] == "UNSUPPORTED"
    layer.close()


def test_expert_path_settings_and_errors(api):
    cfg = wl.with_tokens(wl.CONFIGS["bert"], 64)
    layer = api.Layer.from_config(cfg, wl.make_weights(cfg))
    assert layer.get_expert_path()[:2] == ("auto", 8)
    layer.set_expert_path("gather", group=4, rho_max=0.25)
    assert layer.get_expert_path() == ("gather", 4, 0.25)
    for bad_group in (3, 16, 5):                               # not a divisor of 32 and E, or wider than one MMA
        with pytest.raises(api.D2DError) as e:
            layer.set_expert_path("auto", group=bad_group)
        assert api.STATUS_NAMES[e.value.code] == "UNSUPPORTED"
    layer.reset_counters()
    torch.cuda.synchronize()
    layer.close()
    # the host-side copy of the rule the kernels evaluate: small batches stay dense at any density, large ones go from
    # the fused kernel (plain layers) through the gathered pair to the dense pair as the density grows
    paper = wl.CONFIGS["paper"]
    lp = api.Layer.from_config(paper, wl.make_weights(paper))
    pairs = paper.T * paper.E
    taken = [lp.expert_path_for(paper.T, int(rho * pairs)) for rho in (0.01, 0.05, 0.1, 0.3, 0.6, 1.0)]
    assert taken == ["fused", "fused", "gather", "gather", "dense", "dense"]
    assert all(lp.expert_path_for(2048, int(rho * 2048 * paper.E)) == "dense" for rho in (0.01, 0.3, 1.0))
    for forced in ("dense", "gather", "fused"):
        lp.set_expert_path(forced)
        assert lp.expert_path_for(paper.T, pairs // 2) == forced
    lp.close()
    tiny = wl.CONFIGS["tiny"]                                  # fp32 layers have no tensor-core expert path
    lt = api.Layer.from_config(tiny, wl.make_weights(tiny))
    assert lt.get_expert_path()[1] == 0
    with pytest.raises(api.D2DError) as e:
        lt.set_expert_path("gather")
    assert api.STATUS_NAMES[e.value.code] == "UNSUPPORTED"
    lt.close()


def test_decode_batch_with_truncated_lists_stays_inside_its_buffers(api):
    """A perm buffer smaller than the number of selected pairs: the selection reports D2D_ERR_CAPACITY and the decode
    expert kernel, which walks the lists, must not read past the buffer; guard words behind it stay untouched."""
    cfg = wl.with_tokens(wl.CONFIGS["gpt2_ffn"], 4)
    w, x = wl.make_weights(cfg), wl.make_tokens(cfg)
    layer = api.Layer.from_config(cfg, w)
    cap = 16
    r = layer.new_routing(4, perm_capacity=cap)
    guard = torch.full((4096,), -7, dtype=torch.int32, device="cuda")      # allocated right after: poison would be used as tokens
    y = torch.zeros((4, cfg.d), dtype=torch.bfloat16, device="cuda")
    layer.layer_fwd(api.to_device(x, cfg.dtype), 0.2, y=y, routing=r)
    torch.cuda.synchronize()
    assert r.status == 7 and r.n_sel > cap
    assert bool((guard == -7).all())
    assert torch.isfinite(y.float()).all()
    layer.close()


# (workload, tokens, experts per group or 0 = default, d or 0 = the workload's, densities)
FUSED_CASES = [
    ("bert", 700, 0, 0, (0.0, 0.03, 0.3, 1.0)),     # s = 24, g = 4: 96-column groups, two H k-blocks, the second half full
    ("bert", 1024, 2, 0, (0.2,)),                   # 48-column groups: one H k-block
    ("bert", 333, 0, 464, (0.15,)),                 # d = 464: ragged last k-block of the up projection, ragged last output chunk
    ("vit", 900, 0, 0, (0.05, 0.5)),                # s = 16, g = 8
    ("vit", 600, 1, 0, (0.1,)),                     # one expert per group: 16-column groups
    ("paper", 1500, 0, 0, (0.02, 0.4)),             # s = 128, g = 1
    ("gpt2_attn", 520, 0, 0, (0.1,)),               # d_ff = 2 d: the accumulator fills the whole of H's place
]


@pytest.mark.parametrize("name,T,g,d,ps", FUSED_CASES)
def test_fused_gathered_step_equals_oracle(api, name, T, g, d, ps):
    """The fused kernel (up projection, activation, down projection and merge per group and tile of the tokens that
    keep it; Listing 1 with the atomic merge of App. C) forced through d2d_layer_set_expert_path: y against the
    oracle on the same mask, twice in a row (the counters reset themselves, the accumulator is re-filled), with the
    workspace poisoned before each call."""
    import dataclasses
    cfg = wl.with_tokens(wl.CONFIGS[name], T)
    if d:
        cfg = dataclasses.replace(cfg, d=d)
    w, x = wl.make_weights(cfg), wl.make_tokens(cfg)
    layer = api.Layer.from_config(cfg, w)
    layer.set_expert_path("fused", group=g)
    path, gg, _ = layer.get_expert_path()
    assert path == "fused" and gg >= 1 and gg * cfg.s <= 128 and (g == 0 or gg == g)
    xd = api.to_device(x, cfg.dtype)
    act = oracle.ACT_BY_NAME[cfg.act]
    ws = layer.workspace(T)                                    # the buffer the binding passes to every call
    for p in ps:
        G = _structured_mask(cfg, T, p, seed=29) if 0.0 < p < 1.0 else np.full((T, cfg.E), int(p), np.uint8)
        r = _routing(api, G, cfg.E)
        y_ref = oracle.moe_ffn(x, w["w1"], w["b1"], w["w_gate"], w["w2"], w["b2"], act, G)
        for rep in range(2):
            ws.fill_(0xc1)                                     # float32 0xc1c1c1c1 = -24.2: a stale accumulator would show
            y = torch.full((T, cfg.d), float("nan"), dtype=torch.bfloat16, device="cuda")
            layer.moe_ffn_fwd(xd, r, y=y)
            torch.cuda.synchronize()
            assert r.status == 0
            yg = y.float().cpu().numpy()
            assert np.isfinite(yg).all()
            assert _rel_err(yg, y_ref) <= TOL_Y, (name, p, rep, _rel_err(yg, y_ref))
            assert _per_token_err(yg, y_ref) <= 4 * TOL_Y, (name, p, rep, _per_token_err(yg, y_ref))
        # a token that keeps nothing gets b2 exactly (the accumulator's fill, converted)
        if 0.0 < p < 1.0:
            b2 = torch.from_numpy(np.asarray(w["b2"], np.float32)).to(torch.bfloat16).float().numpy() if w["b2"] is not None else 0.0
            assert np.array_equal(yg[T // 3], np.broadcast_to(b2, (cfg.d,)))
    # gated layers and groups of more than 128 neurons are refused
    with pytest.raises(api.D2DError):
        layer.set_expert_path("fused", group=64)
    layer.close()
