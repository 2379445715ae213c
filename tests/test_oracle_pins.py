"""Pins for the CPU oracle: everything here checks oracle/ against something other than itself.

Sources of truth used: hand-worked fixtures (tests/golden), float64 library routines
(torch matmul / erf / tanh / silu), invariants the paper fixes (Eq. 4, Sec. 3.2), and the
closed-form cost ratio of App. B.
"""
import json
import math
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2310_04361_b200 import workloads as wl

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _gold(name):
    with open(os.path.join(GOLD, name)) as f:
        return json.load(f)


def _a(v, dt=np.float32):
    return np.array(v, dtype=dt)


# ---------------------------------------------------------------- hand-worked fixtures

def test_select_hand_cases():
    g = _gold("select_hand.json")
    R = _a(g["R"])
    for case in g["cases"]:
        G, k, bad = oracle.select(R, case["tau"])
        assert bad == 0
        assert G.tolist() == case["G"], case["tau"]
        assert k.tolist() == case["k"]


def test_metadata_hand_case():
    g = _gold("select_hand.json")
    G, _, _ = oracle.select(_a(g["R"]), 0.5)
    m = oracle.metadata(G)
    want = g["metadata_at_tau_0.5"]
    for key in ("counts", "offsets", "perm", "tok_off", "tok_exp"):
        assert m[key].tolist() == want[key], key
    assert m["n_sel"] == 11


def test_ffn_hand_cases():
    g = _gold("ffn_hand.json")
    x, w1, b1, w2, b2 = (_a(g[k]) for k in ("x", "w1", "b1", "w2", "b2"))
    p = g["plain"]
    ones, none = np.ones((2, 2), np.uint8), np.zeros((2, 2), np.uint8)
    e0 = np.array([[1, 0], [1, 0]], np.uint8)
    e1 = np.array([[0, 1], [0, 1]], np.uint8)
    f = lambda G: oracle.moe_ffn(x, w1, b1, None, w2, b2, oracle.ACT_RELU, G)
    assert f(ones).tolist() == p["y_all"]
    assert f(e0).tolist() == p["y_expert0_only"]
    assert f(e1).tolist() == p["y_expert1_only"]
    assert f(none).tolist() == p["y_none"]
    assert oracle.dense_ffn(x, w1, b1, None, w2, b2, oracle.ACT_RELU).tolist() == p["y_all"]
    norms = oracle.expert_norms(x, w1, b1, None, w2, oracle.ACT_RELU, 2)
    np.testing.assert_allclose(norms ** 2, _a(p["norms_squared"], np.float64), rtol=1e-14)
    # a mask that differs per token picks the per-token rows
    mixed = np.array([[1, 0], [0, 1]], np.uint8)
    assert f(mixed).tolist() == [p["y_expert0_only"][0], p["y_expert1_only"][1]]


def test_gated_ffn_hand_cases():
    g = _gold("ffn_hand.json")
    x, w1, b1, w2, b2, wg = (_a(g[k]) for k in ("x", "w1", "b1", "w2", "b2", "w_gate"))
    p = g["gated"]
    ones = np.ones((2, 2), np.uint8)
    e0 = np.array([[1, 0], [1, 0]], np.uint8)
    assert oracle.moe_ffn(x, w1, b1, wg, w2, b2, oracle.ACT_RELU, ones).tolist() == p["y_all"]
    assert oracle.moe_ffn(x, w1, b1, wg, w2, b2, oracle.ACT_RELU, e0).tolist() == p["y_expert0_only"]
    assert oracle.dense_ffn(x, w1, b1, wg, w2, b2, oracle.ACT_RELU).tolist() == p["y_all"]


def test_router_hand_case():
    r = _gold("ffn_hand.json")["router"]
    R = oracle.router(_a(r["x"]), _a(r["w_r1"]), _a(r["b_r1"]), _a(r["w_r2"]), _a(r["b_r2"]))
    assert R.tolist() == r["R"]


# ---------------------------------------------------------------- library routines (float64)

def _t(a):
    return None if a is None else torch.from_numpy(np.asarray(a, dtype=np.float64))


def _torch_act(z, act):
    if act == "relu":
        return torch.relu(z)
    if act == "gelu_erf":
        return torch.nn.functional.gelu(z)
    if act == "gelu_tanh":
        return torch.nn.functional.gelu(z, approximate="tanh")
    return torch.nn.functional.silu(z)


def _torch_dense(x, w, act):
    x = _t(x)
    up = x @ _t(w["w1"]).T
    if w["b1"] is not None:
        up = up + _t(w["b1"])
    if w["w_gate"] is not None:
        h = _torch_act(x @ _t(w["w_gate"]).T, act) * up
    else:
        h = _torch_act(up, act)
    y = h @ _t(w["w2"]).T
    if w["b2"] is not None:
        y = y + _t(w["b2"])
    return y.numpy()


SMALL = {
    "tiny": wl.CONFIGS["tiny"],
    "gelu": wl.LayerConfig("gelu", "bf16", d=96, d_ff=240, E=10, d_h=16, act="gelu_erf", T=37,
                           token_sigma=0.7, b1_shift=-0.3, seed=11),
    "gelu_tanh": wl.LayerConfig("gelu_tanh", "bf16", d=80, d_ff=144, E=6, d_h=24, act="gelu_tanh", T=19,
                                token_sigma=0.5, b1_shift=-0.2, seed=12),
    "swiglu": wl.LayerConfig("swiglu", "bf16", d=72, d_ff=160, E=5, d_h=8, act="silu", T=23, gated=True,
                             token_sigma=0.7, b1_shift=None, has_b2=False, seed=13),
}


@pytest.mark.parametrize("name", list(SMALL))
def test_router_matches_library_matmul(name):
    cfg = SMALL[name]
    w, x = wl.make_weights(cfg), wl.make_tokens(cfg)
    want = torch.abs(torch.relu(_t(x) @ _t(w["w_r1"]).T + _t(w["b_r1"])) @ _t(w["w_r2"]).T + _t(w["b_r2"]))
    got = oracle.router(x, w["w_r1"], w["b_r1"], w["w_r2"], w["b_r2"])
    assert got.dtype == np.float32
    np.testing.assert_allclose(got, want.numpy(), rtol=2e-7, atol=1e-12)
    # abs on the output: negating the second layer changes nothing (Sec. 3.3)
    flipped = oracle.router(x, w["w_r1"], w["b_r1"], -w["w_r2"], -w["b_r2"])
    assert np.array_equal(flipped, got)
    assert (got >= 0).all()


@pytest.mark.parametrize("name", list(SMALL))
def test_dense_ffn_matches_library_matmul(name):
    cfg = SMALL[name]
    w, x = wl.make_weights(cfg), wl.make_tokens(cfg)
    got = oracle.dense_ffn(x, w["w1"], w["b1"], w["w_gate"], w["w2"], w["b2"], oracle.ACT_BY_NAME[cfg.act])
    want = _torch_dense(x, w, cfg.act)
    np.testing.assert_allclose(got, want, rtol=1e-11, atol=1e-13)


# ---------------------------------------------------------------- invariants the paper fixes

@pytest.mark.parametrize("name", list(SMALL))
def test_tau_zero_reproduces_dense_ffn(name):
    """Sec. 3.2: experts partition the neurons and b2 is shared, so keeping all experts is the dense FFN."""
    cfg = SMALL[name]
    w, x = wl.make_weights(cfg), wl.make_tokens(cfg)
    out = oracle.layer(x, w, oracle.ACT_BY_NAME[cfg.act], 0.0)
    assert out["G"].all() and (out["k"] == cfg.E).all()
    np.testing.assert_allclose(out["y"], _torch_dense(x, w, cfg.act), rtol=1e-11, atol=1e-13)


@pytest.mark.parametrize("name", list(SMALL))
def test_expert_outputs_are_additive(name):
    """y(A u B) - b2 = (y(A) - b2) + (y(B) - b2) for disjoint masks; single experts sum to the FFN."""
    cfg = SMALL[name]
    act = oracle.ACT_BY_NAME[cfg.act]
    w, x = wl.make_weights(cfg), wl.make_tokens(cfg)
    b2 = np.zeros(cfg.d) if w["b2"] is None else w["b2"].astype(np.float64)
    f = lambda G: oracle.moe_ffn(x, w["w1"], w["b1"], w["w_gate"], w["w2"], w["b2"], act, G) - b2
    rng = np.random.default_rng(5)
    A = (rng.random((cfg.T, cfg.E)) < 0.4).astype(np.uint8)
    B = ((rng.random((cfg.T, cfg.E)) < 0.5) & (A == 0)).astype(np.uint8)
    np.testing.assert_allclose(f(A | B), f(A) + f(B), rtol=1e-10, atol=1e-13)
    total = np.zeros((cfg.T, cfg.d))
    norms = oracle.expert_norms(x, w["w1"], w["b1"], w["w_gate"], w["w2"], act, cfg.E)
    for e in range(cfg.E):
        one = np.zeros((cfg.T, cfg.E), np.uint8)
        one[:, e] = 1
        ye = f(one)
        total += ye
        np.testing.assert_allclose(np.linalg.norm(ye, axis=1), norms[:, e], rtol=1e-10, atol=1e-14)
    np.testing.assert_allclose(total + b2, _torch_dense(x, w, cfg.act), rtol=1e-10, atol=1e-12)
    # empty mask: exactly b2
    y0 = oracle.moe_ffn(x, w["w1"], w["b1"], w["w_gate"], w["w2"], w["b2"], act, np.zeros_like(A))
    assert np.array_equal(y0, np.broadcast_to(b2, y0.shape))


def test_relu_positive_homogeneity():
    """With zero biases a ReLU expert block is positively homogeneous: y(a x) = a y(x) for a fixed mask."""
    cfg = wl.LayerConfig("h", "f32", d=48, d_ff=96, E=6, d_h=8, act="relu", T=9, b1_shift=None, has_b2=False, seed=3)
    w, x = wl.make_weights(cfg), wl.make_tokens(cfg)
    G = wl.make_bernoulli_mask(cfg, 0.5)
    f = lambda xx: oracle.moe_ffn(xx, w["w1"], None, None, w["w2"], None, oracle.ACT_RELU, G)
    np.testing.assert_allclose(f(4.0 * x), 4.0 * f(x), rtol=1e-13)


@pytest.mark.parametrize("E", [4, 16, 33, 128, 344])
def test_selection_invariants(E):
    rng = np.random.default_rng(E)
    T = 65
    R = np.abs(rng.standard_normal((T, E))).astype(np.float32)
    R[3] = 0.0                      # all-zero row keeps everything
    R[5, :] = R[5, 0]               # full tie row
    R[7, 1] = R[7].max()            # duplicated maximum
    R[7, E - 1] = R[7].max()
    prev = None
    for tau in (0.0, 0.1, 0.37, 0.5, 0.9, 1.0):
        G, k, bad = oracle.select(R, tau)
        assert bad == 0
        assert (k >= 1).all()                       # the maximum always passes (Eq. 4)
        assert np.array_equal(k, G.sum(1))
        if prev is not None:
            assert (G <= prev).all()                # raising tau only removes experts
        prev = G
        # exact invariance under power-of-two scaling of R
        for j in (-3, 5):
            G2, _, _ = oracle.select(np.ldexp(R, j), tau)
            assert np.array_equal(G2, G)
        # relabelling the experts relabels the mask
        perm = rng.permutation(E)
        Gp, _, _ = oracle.select(np.ascontiguousarray(R[:, perm]), tau)
        assert np.array_equal(Gp, G[:, perm])
    G0, _, _ = oracle.select(R, 0.0)
    assert G0.all()
    G1, _, _ = oracle.select(R, 1.0)
    assert np.array_equal(G1, (R == R.max(1, keepdims=True)).astype(np.uint8))
    assert G1[7, 1] and G1[7, E - 1] and G1[5].all() and G1[3].all()


def test_selection_threshold_is_a_float32_product():
    """Eq. 4's threshold tau*max is ONE float32 round-to-nearest product, compared in float32.

    The pairs below are chosen so that the float32 product lies strictly BELOW the exact real product tau*m (with
    tau itself taken as the float32 value the rule receives): a score equal to the float32 product must then be kept,
    whereas a rule that multiplied in double precision (or in exact arithmetic) would drop it, because it sits under
    that threshold.  One pair of the other direction (float32 product above the exact one) shows the opposite case:
    the float32 neighbour just below the rounded threshold lies above the exact product and must still be dropped."""
    from fractions import Fraction
    tau = np.float32(0.1)
    below_pairs = []
    for m in np.float32([5.0, 123.456, 1e-3, 7e5]):
        thr32 = np.float32(tau * m)                           # numpy: one float32 multiply, round to nearest
        exact = Fraction(float(tau)) * Fraction(float(m))     # the real-number product of the two float32 inputs
        assert Fraction(float(thr32)) < exact, "pair must have its float32 product below the exact product"
        assert float(thr32) < float(tau) * float(m)           # ... and below the double-precision product as well
        below_pairs.append((m, thr32))
    R = np.array([[m, thr32, np.nextafter(thr32, np.float32(-np.inf))] for m, thr32 in below_pairs], dtype=np.float32)
    G, k, _ = oracle.select(R, float(tau))
    # the maximum, the score ON the float32 threshold (kept: >= in float32), the float32 value just under it (dropped)
    assert G.tolist() == [[1, 1, 0]] * len(below_pairs)
    assert k.tolist() == [2] * len(below_pairs)
    # the other direction: float32 product above the exact one
    m = np.float32(3.0)
    thr32 = np.float32(tau * m)
    assert Fraction(float(thr32)) > Fraction(float(tau)) * Fraction(float(m))
    under = np.nextafter(thr32, np.float32(-np.inf))
    assert Fraction(float(under)) < Fraction(float(tau)) * Fraction(float(m))      # no float32 value lies between the two products
    G, _, _ = oracle.select(np.array([[m, thr32, under]], dtype=np.float32), float(tau))
    assert G.tolist() == [[1, 1, 0]]


def test_selection_nonfinite_rows_keep_everything():
    R = np.array([[1.0, np.nan, 0.2], [0.1, 0.5, 0.2], [np.inf, 0.0, 0.0]], dtype=np.float32)
    G, k, bad = oracle.select(R, 0.9)
    assert bad == 1
    assert G.tolist() == [[1, 1, 1], [0, 1, 0], [1, 1, 1]]


def test_brute_force_enumeration_tiny():
    """Every 0/1/2-valued R row of length 3 at tau=0.5 against the rule evaluated in exact rationals."""
    from fractions import Fraction
    rows = [(a, b, c) for a in range(3) for b in range(3) for c in range(3)]
    R = np.array(rows, dtype=np.float32)
    G, k, _ = oracle.select(R, 0.5)
    for row, g in zip(rows, G.tolist()):
        thr = Fraction(1, 2) * max(row)
        assert g == [int(Fraction(v) >= thr) for v in row]


def test_metadata_properties():
    rng = np.random.default_rng(9)
    T, E = 300, 70
    G = (rng.random((T, E)) < 0.3).astype(np.uint8)
    G[17] = 0            # token with nothing ...
    G[:, 5] = 0          # empty expert
    G[:, 6] = 1          # ... except the expert every token keeps
    m = oracle.metadata(G)
    assert m["counts"].sum() == G.sum() == m["n_sel"] == m["offsets"][-1]
    assert m["counts"][5] == 0 and m["counts"][6] == T
    pairs = set()
    for e in range(E):
        bucket = m["perm"][m["offsets"][e]:m["offsets"][e + 1]]
        assert (np.diff(bucket) > 0).all()
        assert np.array_equal(bucket, np.nonzero(G[:, e])[0])   # library nonzero, not the oracle's loop
        pairs.update((int(t), e) for t in bucket)
    dual = set()
    for t in range(T):
        ex = m["tok_exp"][m["tok_off"][t]:m["tok_off"][t + 1]]
        assert np.array_equal(ex, np.nonzero(G[t])[0])
        dual.update((t, int(e)) for e in ex)
    assert pairs == dual
    # closed forms for constructed masks
    ones = oracle.metadata(np.ones((4, 3), np.uint8))
    assert ones["counts"].tolist() == [4, 4, 4] and ones["perm"].tolist() == [0, 1, 2, 3] * 3
    eye = oracle.metadata(np.eye(5, dtype=np.uint8))
    assert eye["perm"].tolist() == [0, 1, 2, 3, 4] and eye["offsets"].tolist() == [0, 1, 2, 3, 4, 5]


def test_mask_packing_layout():
    G = np.zeros((2, 40), np.uint8)
    G[0, 0] = G[0, 31] = G[0, 32] = 1
    G[1, 39] = 1
    m = oracle.pack_mask(G)
    assert m.shape == (2, 2) and m.dtype == np.dtype("<u4")
    assert m.tolist() == [[0x80000001, 0x1], [0, 0x80]]
    assert np.array_equal(oracle.unpack_mask(m, 40), G)


def test_topk_selection():
    R = np.array([[0.5, 0.9, 0.9, 0.1], [0.3, 0.2, 0.1, 0.0]], dtype=np.float32)
    G, k = oracle.select_topk(R, 2)
    assert G.tolist() == [[0, 1, 1, 0], [1, 1, 0, 0]] and k.tolist() == [2, 2]
    G, _ = oracle.select_topk(R, 1)
    assert G.tolist() == [[0, 1, 0, 0], [1, 0, 0, 0]]      # ties go to the lower index
    rng = np.random.default_rng(1)
    R = rng.random((50, 37)).astype(np.float32)
    G, _ = oracle.select_topk(R, 5)
    want = np.zeros_like(G)
    idx = torch.topk(torch.from_numpy(R), 5, dim=1).indices.numpy()   # library top-k, distinct values
    np.put_along_axis(want, idx, 1, axis=1)
    assert np.array_equal(G, want)


# ---------------------------------------------------------------- App. B closed form

@pytest.mark.parametrize("d_m,e,n,d_h", [(768, 4, 128, 128), (768, 4, 192, 128), (1024, 4, 256, 128), (64, 4, 16, 32)])
def test_cost_ratio_closed_form(d_m, e, n, d_h):
    """C_dynk / C_MLP = k/n + d_h (1 + n/d_m) / (2 e d_m)   (App. B)."""
    c_router, c_expert, c_dense = oracle.cost_units(d_m, e * d_m, n, d_h)
    assert c_dense == 2 * e * d_m * d_m
    for k in (1, n // 4, n):
        ratio = (k * c_expert + c_router) / c_dense
        closed = k / n + d_h * (1 + n / d_m) / (2 * e * d_m)
        assert math.isclose(ratio, closed, rel_tol=1e-12)
    if d_m == 6 * d_h and n == 128:       # the paper's setting d_m = 6 d_h, e = 4
        assert math.isclose((c_router) / c_dense, 0.024305555555555556, rel_tol=1e-12)


# ---------------------------------------------------------------- 8-bit expert weights (App. C: narrower formats)

def test_e4m3_table_against_the_format_and_a_library_cast():
    """The 127 finite values: smallest subnormal 2^-9, smallest normal 2^-6, largest 448, eight codes per binade with
    a spacing that doubles from binade to binade; and code for code what torch's float8_e4m3fn holds."""
    v = oracle.e4m3_values()
    assert len(v) == 127 and v[0] == 0.0 and v[1] == 2.0 ** -9 and v[8] == 2.0 ** -6 and v[126] == 448.0
    assert (np.diff(v) > 0).all()
    steps = np.diff(v)
    assert (steps[:15] == 2.0 ** -9).all()                           # subnormals and the first binade share one step
    for b in range(2, 15):                                           # binade b starts at code 8 b
        assert (steps[8 * b: 8 * b + 7] == 2.0 ** (b - 10)).all()
    lib = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).float().numpy()
    codes = np.arange(256, dtype=np.uint8)
    finite = (codes & 0x7F) != 0x7F
    assert np.array_equal(oracle.e4m3_decode(codes[finite]), lib[finite].astype(np.float64))


def test_e4m3_rounding_is_to_nearest_with_ties_to_even_and_saturates():
    # hand-placed ties: halfway between two neighbours the code with an even mantissa bit wins
    x = np.array([2.0 ** -10, 3 * 2.0 ** -10, 1.0625, 1.1875, 17.0, 19.0, -17.0, 432.0])
    assert oracle.e4m3_encode(x).tolist() == [0, 2, 56, 58, 88, 90, 0x80 | 88, 126]
    # just off the tie the nearer neighbour wins
    assert oracle.e4m3_encode(np.array([1.0625 + 1e-9, 1.0625 - 1e-9])).tolist() == [57, 56]
    # beyond the largest finite value: saturation, never the NaN code
    assert oracle.e4m3_encode(np.array([449.0, 1e9, -1e9])).tolist() == [126, 126, 0x80 | 126]
    # every representable value encodes to itself
    codes = np.array([c for c in range(256) if (c & 0x7F) != 0x7F and c != 0x80], dtype=np.uint8)
    assert np.array_equal(oracle.e4m3_encode(oracle.e4m3_decode(codes)), codes)
    # a library cast agrees on random in-range values (torch rounds to nearest even as well)
    rng = np.random.default_rng(5)
    r = (rng.standard_normal(20000) * np.exp(rng.uniform(-8, 5, 20000))).astype(np.float32)
    r = r[np.abs(r) <= 448.0]
    lib = torch.from_numpy(r).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    ours = oracle.e4m3_encode(r)
    zero = (ours & 0x7F) == 0                                        # the sign of a value rounded to zero is free
    assert np.array_equal(ours[~zero], lib[~zero]) and ((lib[zero] & 0x7F) == 0).all()


def test_expert_scales_are_the_smallest_power_of_two_that_fits():
    rng = np.random.default_rng(8)
    E, s, d = 6, 8, 32
    w = (rng.standard_normal((E * s, d)) * 0.02).astype(np.float32)
    w[2 * s: 3 * s] = 0.0                                            # an all-zero expert
    w[3 * s: 4 * s] *= 0.0
    w[3 * s, 0] = 448.0 * 2.0 ** -9                                  # an expert whose maximum sits exactly on the boundary
    w[4 * s: 5 * s] *= 1e3
    codes, k, deq = oracle.quantize_experts_e4m3(w, E)
    assert k[2] == 0 and not codes[2 * s: 3 * s].any()
    assert k[3] == -9 and codes[3 * s, 0] == 126
    for e in range(E):
        blk = np.abs(w[e * s: (e + 1) * s].astype(np.float64))
        if blk.max() > 0:
            assert blk.max() <= 448.0 * 2.0 ** int(k[e]) < 2 * blk.max()        # fits, and half the scale would not
        # error of a normal value: half a mantissa step, 2^-4 relative; below the smallest normal: 2^(k - 10) absolute
        err = np.abs(deq[e * s: (e + 1) * s].astype(np.float64) - w[e * s: (e + 1) * s])
        assert (err <= np.maximum(blk * 2.0 ** -4, 2.0 ** (int(k[e]) - 10))).all()
    # the dequantised weights are bfloat16 values: a layer can hold them in its bf16 copies without further rounding
    assert torch.equal(torch.from_numpy(deq).to(torch.bfloat16).float(), torch.from_numpy(deq))
    # scaling an expert by a power of two moves its exponent and leaves its codes alone
    w2 = w.copy(); w2[: s] *= 4.0
    codes2, k2, _ = oracle.quantize_experts_e4m3(w2, E)
    assert k2[0] == k[0] + 2 and np.array_equal(codes2[: s], codes[: s])
