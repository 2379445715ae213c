"""Seeded synthetic inputs shaped like the paper's BERT / ViT / GPT-2 / Llama-style layers.

This module holds no arithmetic of the method: it only draws random tensors
(numpy PCG64, float32) and, for bf16 workloads, rounds them once to
bf16-representable float32 values so that the CPU oracle and the CUDA library
consume bit-identical inputs.  It imports neither of them.

No dataset or checkpoint is involved.  The tensors stand in for the paper's
ViT-B/ImageNet, BERT/CARER, GPT-2/OpenWebText and Gemma/C4 layers by shape only
(Sec. 4, App. H); the weight and input distributions are the ones the workload
descriptions state.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace

import numpy as np


@dataclass(frozen=True)
class LayerConfig:
    name: str
    dtype: str            # "f32" | "bf16"
    d: int                # model width
    d_ff: int             # FFN hidden width = E * s
    E: int                # number of experts
    d_h: int              # router hidden width
    act: str              # "relu" | "gelu_erf" | "gelu_tanh" | "silu"
    T: int                # tokens
    gated: bool = False
    token_sigma: float = 0.0     # per-token scale exp(N(0, sigma^2)); 0 = none
    b1_shift: float | None = None  # constant first-layer bias; None = no b1
    has_b2: bool = True
    seed: int = 0
    taus: tuple = ()

    @property
    def s(self) -> int:
        return self.d_ff // self.E

    @property
    def n_mat(self) -> int:
        return 3 if self.gated else 2


def _shift(q: float, d: int) -> float:
    """Bias that leaves a fraction q of N(0, 0.02^2 d) pre-activations negative (q-quantile shift)."""
    z = {0.8: 0.8416212335729143, 0.9: 1.2815515655446004}[q]
    return -z * 0.02 * math.sqrt(d)


CONFIGS = {
    # tiny fp32 case the oracle finishes instantly
    "tiny": LayerConfig("tiny", "f32", d=64, d_ff=256, E=16, d_h=32, act="relu", T=128,
                        token_sigma=0.5, b1_shift=-0.05, seed=0, taus=(0.0, 0.5, 1.0)),
    # BERT-base-shaped: 32 sequences x 128 tokens
    "bert": LayerConfig("bert", "bf16", d=768, d_ff=3072, E=128, d_h=128, act="gelu_erf", T=32 * 128,
                        token_sigma=0.7, b1_shift=_shift(0.8, 768), seed=2,
                        taus=(0.05, 0.1, 0.2, 0.3, 0.5, 0.7, 0.9)),
    # ViT-B/16-shaped: batch 128 x 197 tokens
    "vit": LayerConfig("vit", "bf16", d=768, d_ff=3072, E=192, d_h=128, act="gelu_erf", T=128 * 197,
                       token_sigma=0.0, b1_shift=_shift(0.9, 768), seed=3, taus=(0.1, 0.3, 0.6)),
    # GPT-2-medium-shaped decode FFN; T is overridden with 1, 8, 64
    "gpt2_ffn": LayerConfig("gpt2_ffn", "bf16", d=1024, d_ff=4096, E=256, d_h=128, act="gelu_erf", T=64,
                            token_sigma=0.5, b1_shift=_shift(0.8, 1024), seed=4, taus=(0.2, 0.5)),
    # MoE-fied attention projection d -> 2d -> d on the same tokens
    "gpt2_attn": LayerConfig("gpt2_attn", "bf16", d=1024, d_ff=2048, E=128, d_h=128, act="gelu_erf", T=64,
                             token_sigma=0.5, b1_shift=_shift(0.8, 1024), seed=4, taus=(0.2, 0.5)),
    # Llama-style gated FFN, no biases
    "llama": LayerConfig("llama", "bf16", d=4096, d_ff=11008, E=344, d_h=256, act="silu", T=8192,
                         gated=True, token_sigma=0.7, b1_shift=None, has_b2=False, seed=5,
                         taus=(0.1, 0.2, 0.4, 0.6, 0.8)),
    # the paper's own latency benchmark shape (Sec. 4.4): 24 experts x 128 neurons, 256 x 197 tokens
    "paper": LayerConfig("paper", "bf16", d=768, d_ff=3072, E=24, d_h=128, act="gelu_erf", T=256 * 197,
                         token_sigma=0.0, b1_shift=_shift(0.8, 768), seed=6, taus=()),
}


def with_tokens(cfg: LayerConfig, T: int) -> LayerConfig:
    return replace(cfg, T=int(T))


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round float32 to the nearest bf16 value (ties to even), returned as float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(a.shape)


def _finish(a: np.ndarray, dtype: str) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float32)
    return round_to_bf16(a) if dtype == "bf16" else a


def make_weights(cfg: LayerConfig) -> dict:
    """Layer parameters in nn.Linear layout [out, in]; absent biases are None."""
    rng = np.random.Generator(np.random.PCG64(cfg.seed * 1000 + 1))
    dt = cfg.dtype

    def normal(shape, std):
        return _finish(rng.standard_normal(shape, dtype=np.float32) * np.float32(std), dt)

    w = {
        "w_r1": normal((cfg.d_h, cfg.d), 1.0 / math.sqrt(cfg.d)),
        "b_r1": normal((cfg.d_h,), 0.1),
        "w_r2": normal((cfg.E, cfg.d_h), 1.0 / math.sqrt(cfg.d_h)),
        "b_r2": normal((cfg.E,), 0.1),
        "w1": normal((cfg.d_ff, cfg.d), 0.02),
        "b1": None if cfg.b1_shift is None else _finish(np.full((cfg.d_ff,), cfg.b1_shift, np.float32), dt),
        "w_gate": normal((cfg.d_ff, cfg.d), 0.02) if cfg.gated else None,
        "w2": normal((cfg.d, cfg.d_ff), 0.02),
        "b2": normal((cfg.d,), 0.02) if cfg.has_b2 else None,
    }
    return w


def make_tokens(cfg: LayerConfig, T: int | None = None, stream: int = 0) -> np.ndarray:
    """x [T, d]: N(0,1) entries times a per-token lognormal scale; `stream` selects an independent batch."""
    T = cfg.T if T is None else int(T)
    rng = np.random.Generator(np.random.PCG64(cfg.seed * 1000 + 7 + 13 * stream))
    x = rng.standard_normal((T, cfg.d), dtype=np.float32)
    if cfg.token_sigma > 0:
        scale = np.exp(rng.standard_normal((T, 1), dtype=np.float32) * np.float32(cfg.token_sigma))
        x = x * scale
    return _finish(x, cfg.dtype)


def make_bernoulli_mask(cfg: LayerConfig, p: float, T: int | None = None, stream: int = 0) -> np.ndarray:
    """Override mask of the paper's latency protocol (Sec. 4.4): G[t,e] ~ Bernoulli(p), uint8 [T,E]."""
    T = cfg.T if T is None else int(T)
    rng = np.random.Generator(np.random.PCG64(cfg.seed * 1000 + 101 + 13 * stream))
    return (rng.random((T, cfg.E)) < p).astype(np.uint8)


def make_router_scores(cfg: LayerConfig, T: int | None = None, stream: int = 0) -> np.ndarray:
    """A stand-alone non-negative score matrix [T,E] (half-normal) for selection-only tests."""
    T = cfg.T if T is None else int(T)
    rng = np.random.Generator(np.random.PCG64(cfg.seed * 1000 + 211 + 13 * stream))
    return np.abs(rng.standard_normal((T, cfg.E), dtype=np.float32))
