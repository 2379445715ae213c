"""ctypes front end of the CPU oracle (oracle/d2d_oracle.c).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's CPU
baseline may import this package; the CUDA library and its Python binding never
do.  Nothing here shares code with the CUDA path.  Arrays are numpy; floating
point inputs are float32 (bf16 workloads hold bf16-representable float32
values), outputs are float64 except the router output R (float32, because the
selection rule is taken on the float32 R).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "d2d_oracle.c")
_LIB = os.path.join(_HERE, "libd2d_oracle.so")

ACT_RELU, ACT_GELU_ERF, ACT_GELU_TANH, ACT_SILU = 0, 1, 2, 3
ACT_BY_NAME = {"relu": ACT_RELU, "gelu_erf": ACT_GELU_ERF, "gelu_tanh": ACT_GELU_TANH, "silu": ACT_SILU}


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no FMA contraction) and return the .so path."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared",
               "-Wall", "-Wextra", _SRC, "-o", _LIB, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
    return _lib


def _f32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float32)


def _p(a, ctype=ctypes.c_float):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ctype))


def num_threads() -> int:
    lib = _load()
    lib.d2d_oracle_num_threads.restype = ctypes.c_int
    return int(lib.d2d_oracle_num_threads())


def set_num_threads(n: int) -> None:
    _load().d2d_oracle_set_num_threads(ctypes.c_int(int(n)))


def router(x, w_r1, b_r1, w_r2, b_r2) -> np.ndarray:
    """R[t,i] = |b_r2 + W_r2 relu(b_r1 + W_r1 x_t)|, float32 [T,E] (Sec. 3.3)."""
    x, w_r1, b_r1, w_r2, b_r2 = map(_f32, (x, w_r1, b_r1, w_r2, b_r2))
    T, d = x.shape
    d_h, E = w_r1.shape[0], w_r2.shape[0]
    assert w_r1.shape == (d_h, d) and w_r2.shape == (E, d_h)
    R = np.empty((T, E), dtype=np.float32)
    _load().d2d_oracle_router(_p(x), T, d, _p(w_r1), _p(b_r1), d_h, _p(w_r2), _p(b_r2), E, _p(R))
    return R


def select(R, tau: float):
    """Dynamic-k rule (Eq. 4). Returns (G uint8 [T,E], k int32 [T], nonfinite flag)."""
    R = _f32(R)
    T, E = R.shape
    G = np.empty((T, E), dtype=np.uint8)
    k = np.empty((T,), dtype=np.int32)
    bad = ctypes.c_int32(0)
    _load().d2d_oracle_select(_p(R), T, E, ctypes.c_float(tau), _p(G, ctypes.c_uint8),
                              _p(k, ctypes.c_int32), ctypes.byref(bad))
    return G, k, int(bad.value)


def select_topk(R, kk: int):
    """Static top-k selection, ties to the lower expert index. Returns (G, k)."""
    R = _f32(R)
    T, E = R.shape
    G = np.empty((T, E), dtype=np.uint8)
    k = np.empty((T,), dtype=np.int32)
    _load().d2d_oracle_select_topk(_p(R), T, E, int(kk), _p(G, ctypes.c_uint8), _p(k, ctypes.c_int32))
    return G, k


def metadata(G) -> dict:
    """counts, offsets, perm (expert-major token lists), tok_off, tok_exp (token-major dual)."""
    G = np.ascontiguousarray(G, dtype=np.uint8)
    T, E = G.shape
    n_sel = int(G.sum())
    counts = np.empty((E,), dtype=np.int32)
    offsets = np.empty((E + 1,), dtype=np.int32)
    perm = np.empty((max(n_sel, 1),), dtype=np.int32)
    tok_off = np.empty((T + 1,), dtype=np.int32)
    tok_exp = np.empty((max(n_sel, 1),), dtype=np.int32)
    i32 = ctypes.c_int32
    _load().d2d_oracle_metadata(_p(G, ctypes.c_uint8), T, E, _p(counts, i32), _p(offsets, i32),
                                _p(perm, i32), _p(tok_off, i32), _p(tok_exp, i32))
    return {"counts": counts, "offsets": offsets, "perm": perm[:n_sel], "tok_off": tok_off,
            "tok_exp": tok_exp[:n_sel], "n_sel": n_sel}


def pack_mask(G) -> np.ndarray:
    """The mask in the library's boundary layout: uint32 [T, ceil(E/32)], expert i = bit i%32 of word i//32."""
    G = np.ascontiguousarray(G, dtype=np.uint8)
    T, E = G.shape
    W = (E + 31) // 32
    padded = np.zeros((T, W * 32), dtype=np.uint8)
    padded[:, :E] = G
    bits = np.packbits(padded.reshape(T, W, 32), axis=-1, bitorder="little")  # [T,W,4] bytes
    return np.ascontiguousarray(bits).view("<u4").reshape(T, W)


def unpack_mask(mask, E: int) -> np.ndarray:
    mask = np.ascontiguousarray(mask, dtype="<u4")
    T, W = mask.shape
    bits = np.unpackbits(mask.view(np.uint8).reshape(T, W, 4), axis=-1, bitorder="little")
    return np.ascontiguousarray(bits.reshape(T, W * 32)[:, :E])


def _ffn_args(x, w1, b1, w_gate, w2, b2):
    x, w1, b1, w_gate, w2, b2 = map(_f32, (x, w1, b1, w_gate, w2, b2))
    T, d = x.shape
    d_ff = w1.shape[0]
    assert w1.shape == (d_ff, d) and w2.shape == (d, d_ff)
    assert w_gate is None or w_gate.shape == (d_ff, d)
    return x, w1, b1, w_gate, w2, b2, T, d, d_ff


def moe_ffn(x, w1, b1, w_gate, w2, b2, act: int, G) -> np.ndarray:
    """y[t] = b2 + sum over kept experts of W2[:, block] h_block(x_t); float64 [T,d] (Sec. 3.2, 3.4)."""
    x, w1, b1, w_gate, w2, b2, T, d, d_ff = _ffn_args(x, w1, b1, w_gate, w2, b2)
    G = np.ascontiguousarray(G, dtype=np.uint8)
    E = G.shape[1]
    assert G.shape[0] == T and d_ff % E == 0
    y = np.empty((T, d), dtype=np.float64)
    _load().d2d_oracle_moe_ffn(_p(x), T, d, d_ff, E, _p(w1), _p(b1), _p(w_gate), _p(w2), _p(b2),
                               int(act), _p(G, ctypes.c_uint8), _p(y, ctypes.c_double))
    return y


def dense_ffn(x, w1, b1, w_gate, w2, b2, act: int) -> np.ndarray:
    """The original dense FFN, no experts involved; float64 [T,d]."""
    x, w1, b1, w_gate, w2, b2, T, d, d_ff = _ffn_args(x, w1, b1, w_gate, w2, b2)
    y = np.empty((T, d), dtype=np.float64)
    _load().d2d_oracle_dense_ffn(_p(x), T, d, d_ff, _p(w1), _p(b1), _p(w_gate), _p(w2), _p(b2),
                                 int(act), _p(y, ctypes.c_double))
    return y


def expert_norms(x, w1, b1, w_gate, w2, act: int, E: int) -> np.ndarray:
    """||E_i(x_t)||_2, the router's regression target (Eq. 3); float64 [T,E]."""
    x, w1, b1, w_gate, w2, _, T, d, d_ff = _ffn_args(x, w1, b1, w_gate, w2, None)
    out = np.empty((T, E), dtype=np.float64)
    _load().d2d_oracle_expert_norms(_p(x), T, d, d_ff, int(E), _p(w1), _p(b1), _p(w_gate), _p(w2),
                                    int(act), _p(out, ctypes.c_double))
    return out


def cost_units(d: int, d_ff: int, E: int, d_h: int, gated: bool = False):
    """Per-token cost units of App. B (one per weight touched): (router, one expert, dense FFN)."""
    r, e, f = ctypes.c_int64(0), ctypes.c_int64(0), ctypes.c_int64(0)
    _load().d2d_oracle_cost_units(int(d), int(d_ff), int(E), int(d_h), int(bool(gated)),
                                  ctypes.byref(r), ctypes.byref(e), ctypes.byref(f))
    return int(r.value), int(e.value), int(f.value)


def layer(x, wts: dict, act: int, tau: float) -> dict:
    """Whole layer in the paper's order: router -> dynamic-k -> metadata -> experts + combine."""
    R = router(x, wts["w_r1"], wts.get("b_r1"), wts["w_r2"], wts.get("b_r2"))
    G, k, bad = select(R, tau)
    meta = metadata(G)
    y = moe_ffn(x, wts["w1"], wts.get("b1"), wts.get("w_gate"), wts["w2"], wts.get("b2"), act, G)
    return {"R": R, "G": G, "k": k, "nonfinite": bad, "y": y, **meta}


# ---------------------------------------------------------------------------------------------------------
# Low-precision expert weights (the paper's App. C runs the expert kernels on narrower number formats): an
# expert's weights as 8-bit floating point (1 sign, 4 exponent, 3 mantissa bits, bias 7, no infinities: the
# "e4m3" format) with ONE power-of-two scale per expert and matrix.  Written out from the format's definition:
# the 127 finite non-negative values are tabulated and a weight goes to the nearest one, ties to the code with
# an even mantissa bit, values beyond the largest finite one (448) to 448.

def e4m3_values() -> np.ndarray:
    """The value of every non-negative finite code 0x00 .. 0x7e (code 0x7f is NaN), ascending."""
    v = np.empty(127, dtype=np.float64)
    for code in range(127):
        e, m = code >> 3, code & 7
        v[code] = (m / 8.0) * 2.0 ** -6 if e == 0 else (1.0 + m / 8.0) * 2.0 ** (e - 7)
    return v


def e4m3_encode(a) -> np.ndarray:
    """Codes (uint8, sign in bit 7) of the e4m3 values nearest to `a` (float array, finite): round to nearest,
    ties to even, saturating at +-448."""
    a = np.asarray(a, dtype=np.float64)
    vals = e4m3_values()
    mag = np.minimum(np.abs(a), vals[-1])
    hi = np.searchsorted(vals, mag, side="left")              # first code whose value is >= mag
    hi = np.minimum(hi, 126)
    lo = np.maximum(hi - 1, 0)
    d_lo, d_hi = mag - vals[lo], vals[hi] - mag
    take_hi = (d_hi < d_lo) | ((d_hi == d_lo) & (hi % 2 == 0))
    code = np.where(take_hi, hi, lo).astype(np.uint8)
    return code | (np.signbit(a).astype(np.uint8) << 7)


def e4m3_decode(code) -> np.ndarray:
    code = np.asarray(code, dtype=np.uint8)
    v = e4m3_values()[np.minimum(code & 0x7F, 126)]
    return np.where(code & 0x80, -v, v)


def quantize_experts_e4m3(w_rows, n_experts: int):
    """w_rows: [n_experts * s, d] float, expert e owns rows [e*s, (e+1)*s) (W1 or W_gate as given; for W2 pass its
    transpose).  Per expert: scale 2^k with the smallest integer k for which max|w| / 2^k <= 448 (k = 0 for an
    all-zero expert), codes = e4m3_encode(w / 2^k).  Returns (codes uint8 [n_experts*s, d], k int32 [n_experts],
    dequantised float32 [n_experts*s, d] = decode(codes) * 2^k, exactly representable in bfloat16)."""
    w = np.asarray(w_rows, dtype=np.float64)
    rows, d = w.shape
    s = rows // n_experts
    blocks = w.reshape(n_experts, s * d)
    amax = np.abs(blocks).max(axis=1)
    k = np.zeros(n_experts, dtype=np.int32)
    nz = amax > 0
    # smallest k with amax <= 448 * 2^k: frexp gives amax / 448 = f * 2^p with f in [0.5, 1), so k = p unless f == 0.5
    f, p = np.frexp(amax[nz] / 448.0)
    k[nz] = np.where(f == 0.5, p - 1, p)
    scale = np.ldexp(1.0, k)[:, None]
    codes = e4m3_encode(blocks / scale)
    deq = (e4m3_decode(codes) * scale).astype(np.float32)
    return codes.reshape(rows, d), k, deq.reshape(rows, d)
