"""Seeded synthetic attention inputs shaped like the paper's workloads.

This module holds NO arithmetic of the method (no quantizer, no softmax): it only draws
random tensors and rounds them to bf16.  It is the one module shared by the CPU oracle's
tests and by the CUDA path's tests / benchmark, so that both sides see identical bits.

The paper evaluates on Wan2.2-14B (81 frames, 720p) and HunyuanVideo-13B (129 frames,
720p) attention tensors (Section 5.1, "Implementation Details"); those activations are not
available, so the generators below stand in for them with the same shapes and with the
outlier structure that makes 4-bit attention hard (a few large channels, a few large
tokens, a shared low-rank component).

Every head (b, h) is drawn from its own generator ``default_rng([seed, b*H + h])`` in the
order Q, K, V, so a single head can be regenerated without drawing the whole tensor.

bf16 values are carried as ``uint16`` bit patterns (NumPy has no bf16 dtype);
``bf16_bits_to_f32`` widens them exactly.
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np

HEAD_DIM = 128


# ----------------------------------------------------------------------------- bf16 helpers
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to fp32."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


# ----------------------------------------------------------------------------- configs
@dataclasses.dataclass(frozen=True)
class AttnConfig:
    name: str
    B: int
    H: int
    Nq: int
    Nkv: int
    seed: int
    recipe: str  # "iid" | "outlier" | "wan" | "hunyuan"
    d: int = HEAD_DIM

    @property
    def softmax_scale(self) -> float:
        return 1.0 / math.sqrt(self.d)

    @property
    def flops(self) -> float:
        return 4.0 * self.B * self.H * self.Nq * self.Nkv * self.d


CONFIGS = {
    # the four named configurations of the benchmark definition
    "tiny": AttnConfig("tiny", 1, 2, 1024, 1024, 0, "iid"),
    "outlier": AttnConfig("outlier", 1, 24, 8192, 8192, 1, "outlier"),
    "wan22": AttnConfig("wan22", 1, 40, 75600, 75600, 2, "wan"),
    "hunyuan": AttnConfig("hunyuan", 1, 24, 119056, 119056, 3, "hunyuan"),
}
for _n in (4096, 16384, 32768, 65536):  # the N sweep of the benchmark definition
    CONFIGS[f"sweep{_n}"] = AttnConfig(f"sweep{_n}", 1, 40, _n, _n, 100 + int(math.log2(_n)), "outlier")

# Wan2.2 has separate cross-attention modules (paper Section 5.1): video queries against a short text
# context.  512 context tokens stand in for the text encoder's sequence.
CONFIGS["wan22_cross"] = AttnConfig("wan22_cross", 1, 40, 75600, 512, 4, "wan")

HUNYUAN_VIDEO_TOKENS = 118800


def _head_rng(cfg: AttnConfig, b: int, h: int) -> np.random.Generator:
    return np.random.default_rng([cfg.seed, b * cfg.H + h])


def make_head(cfg: AttnConfig, b: int, h: int):
    """Return (q, k, v) of one head as uint16 bf16 bit patterns, shapes [Nq,d], [Nkv,d], [Nkv,d]."""
    rng = _head_rng(cfg, b, h)
    d = cfg.d
    q = rng.standard_normal((cfg.Nq, d), dtype=np.float32)
    k = rng.standard_normal((cfg.Nkv, d), dtype=np.float32)
    v = rng.standard_normal((cfg.Nkv, d), dtype=np.float32)
    if cfg.recipe == "iid":
        pass
    elif cfg.recipe == "outlier":
        # 8 of 128 channels x16 (same channels for Q and K); 1% of tokens x8 (independent draws)
        ch = rng.choice(d, 8, replace=False)
        q[:, ch] *= 16.0
        k[:, ch] *= 16.0
        tq = rng.choice(cfg.Nq, cfg.Nq // 100, replace=False)
        tk = rng.choice(cfg.Nkv, cfg.Nkv // 100, replace=False)
        q[tq, :] *= 8.0
        k[tk, :] *= 8.0
    elif cfg.recipe == "wan":
        # rank-4 component shared by Q and K with E||U w||^2 = 16, then 6 channels x10
        g = rng.standard_normal((d, 4)).astype(np.float64)
        u, _ = np.linalg.qr(g)
        u = u.astype(np.float32)
        wq = rng.standard_normal((cfg.Nq, 4), dtype=np.float32) * np.float32(2.0)
        wk = rng.standard_normal((cfg.Nkv, 4), dtype=np.float32) * np.float32(2.0)
        q += wq @ u.T
        k += wk @ u.T
        ch = rng.choice(d, 6, replace=False)
        q[:, ch] *= 10.0
        k[:, ch] *= 10.0
    elif cfg.recipe == "hunyuan":
        # video tokens: 8 channels x12; text tokens (the tail): variance 2, no outliers
        ch = rng.choice(d, 8, replace=False)
        nvq = min(HUNYUAN_VIDEO_TOKENS, cfg.Nq)
        nvk = min(HUNYUAN_VIDEO_TOKENS, cfg.Nkv)
        q[:nvq, ch] *= 12.0
        k[:nvk, ch] *= 12.0
        q[nvq:, :] *= np.float32(math.sqrt(2.0))
        k[nvk:, :] *= np.float32(math.sqrt(2.0))
    else:
        raise ValueError(cfg.recipe)
    return f32_to_bf16_bits(q), f32_to_bf16_bits(k), f32_to_bf16_bits(v)


def make_all(cfg: AttnConfig):
    """Full (q, k, v) as uint16 arrays of shape [B,H,N,d]."""
    q = np.empty((cfg.B, cfg.H, cfg.Nq, cfg.d), np.uint16)
    k = np.empty((cfg.B, cfg.H, cfg.Nkv, cfg.d), np.uint16)
    v = np.empty((cfg.B, cfg.H, cfg.Nkv, cfg.d), np.uint16)
    for b in range(cfg.B):
        for h in range(cfg.H):
            q[b, h], k[b, h], v[b, h] = make_head(cfg, b, h)
    return q, k, v


def custom_config(name: str, B: int, H: int, Nq: int, Nkv: int, seed: int, recipe: str = "iid") -> AttnConfig:
    return AttnConfig(name, B, H, Nq, Nkv, seed, recipe)


def quantize_sweep_matrix(n_elements: int, seed: int = 7) -> np.ndarray:
    """bf16 N(0,1) matrix [n/128, 128] for the standalone quantize sweep."""
    rng = np.random.default_rng([seed, n_elements])
    return f32_to_bf16_bits(rng.standard_normal((n_elements // HEAD_DIM, HEAD_DIM), dtype=np.float32))
