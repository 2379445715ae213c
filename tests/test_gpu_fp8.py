"""GPU parity of layers with 8-bit (e4m3) expert weights, one power-of-two scale per expert and matrix (the narrower
formats of App. C applied to the expert weights of Sec. 3.2).

The library's codes and exponents must equal the oracle's bit for bit (the rounding of a weight decides an integer
code: both sides take it on the same bf16 weights); y is then compared with the oracle run on the dequantised weights,
on every path of the layer: the decode kernels (which read the codes), the tensor-core kernels (which read the bf16
copy of the dequantised weights), dense and gathered.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2310_04361_b200 import workloads as wl

pytestmark = pytest.mark.gpu

TOL_Y = 2e-2


@pytest.fixture(scope="module")
def api():
    from paper_2310_04361_b200 import api as _api
    assert torch.cuda.is_available()
    return _api


def _rel_err(got, ref):
    ref = np.asarray(ref, dtype=np.float64)
    return float(np.abs(np.asarray(got, dtype=np.float64) - ref).max() / max(np.abs(ref).max(), 1e-30))


def _quantised(cfg, w):
    """The oracle's codes, exponents and dequantised weights of W1, W_gate, W2 (W2 through its transpose)."""
    q = {}
    q["w1"] = oracle.quantize_experts_e4m3(w["w1"], cfg.E)
    q["w_gate"] = oracle.quantize_experts_e4m3(w["w_gate"], cfg.E) if w["w_gate"] is not None else None
    q["w2"] = oracle.quantize_experts_e4m3(np.ascontiguousarray(np.asarray(w["w2"]).T), cfg.E)
    wq = dict(w)
    wq["w1"] = q["w1"][2]
    wq["w_gate"] = q["w_gate"][2] if q["w_gate"] is not None else None
    wq["w2"] = np.ascontiguousarray(q["w2"][2].T)
    return q, wq


@pytest.mark.parametrize("name", ["gpt2_ffn", "bert", "llama"])
def test_codes_and_exponents_equal_the_oracles(api, name):
    cfg = wl.with_tokens(wl.CONFIGS[name], 8)
    w = wl.make_weights(cfg)
    if name == "bert":
        # an all-zero expert, and an expert whose largest weight sits exactly on a scale boundary
        w["w1"][: cfg.s] = 0.0
        w["w1"][cfg.s: 2 * cfg.s] = np.clip(w["w1"][cfg.s: 2 * cfg.s], -0.05, 0.05)
        w["w1"][cfg.s, 0] = 448.0 * 2.0 ** -13
    q, _ = _quantised(cfg, w)
    layer = api.Layer.from_config(cfg, w, fp8_experts=True)
    for which in ("w1", "w_gate", "w2"):
        if q[which] is None:
            with pytest.raises(api.D2DError):
                layer.get_fp8(which)
            continue
        codes, exps = layer.get_fp8(which)
        torch.cuda.synchronize()
        want_codes, want_k, _ = q[which]
        assert np.array_equal(exps.cpu().numpy(), want_k), which
        got = codes.cpu().numpy()
        zero = (want_codes & 0x7F) == 0                      # the sign of a weight that rounds to zero carries nothing
        assert np.array_equal(got[~zero], want_codes[~zero]), which
        assert ((got[zero] & 0x7F) == 0).all()
    layer.close()
    tiny = wl.CONFIGS["tiny"]                                 # float32 layers have no 8-bit form
    with pytest.raises(api.D2DError) as e:
        api.Layer.from_config(tiny, wl.make_weights(tiny), fp8_experts=True)
    assert api.STATUS_NAMES[e.value.code] == "UNSUPPORTED"


FP8_CASES = [("gpt2_ffn", 1, 0.2), ("gpt2_ffn", 3, 0.5), ("gpt2_ffn", 4, 0.2), ("gpt2_attn", 2, 0.2), ("gpt2_ffn", 40, 0.5),
             ("bert", 700, 0.3), ("llama", 2, 0.4), ("llama", 300, 0.4)]


@pytest.mark.parametrize("name,T,tau", FP8_CASES)
def test_layer_with_8bit_experts_matches_the_oracle_on_the_dequantised_weights(api, name, T, tau):
    cfg = wl.with_tokens(wl.CONFIGS[name], T)
    w, x = wl.make_weights(cfg), wl.make_tokens(cfg)
    _, wq = _quantised(cfg, w)
    layer = api.Layer.from_config(cfg, w, fp8_experts=True)
    act = oracle.ACT_BY_NAME[cfg.act]
    xd = api.to_device(x, cfg.dtype)
    for path in (("dense", "gather") if T > 64 else ("auto",)):
        layer.set_expert_path(path)
        y, r = layer.layer_fwd(xd, tau)
        torch.cuda.synchronize()
        assert r.status == 0
        G = oracle.unpack_mask(r.mask_u32(), cfg.E)          # the router is not quantised: the mask is the library's own
        y_ref = oracle.moe_ffn(x, wq["w1"], wq["b1"], wq["w_gate"], wq["w2"], wq["b2"], act, G)
        yg = y.float().cpu().numpy()
        assert np.isfinite(yg).all()
        assert _rel_err(yg, y_ref) <= TOL_Y, (name, T, path, _rel_err(yg, y_ref))
        # and the rounding of the weights is visible: against the unquantised weights the result differs
        y_full = oracle.moe_ffn(x, w["w1"], w["b1"], w["w_gate"], w["w2"], w["b2"], act, G)
        assert _rel_err(y_ref, y_full) > 1e-3
    layer.close()
