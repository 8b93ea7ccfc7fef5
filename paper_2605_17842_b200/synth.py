"""Seeded synthetic inputs: model shapes, random-init weights, stream-mixing matrices, token ids.

This module holds none of the method's arithmetic.  It only produces the inputs that are handed,
byte for byte, to both the CUDA library and the CPU checker used by the tests: numpy float32
arrays (already rounded to bf16-representable values when ``dtype == "bf16"``) and int32 ids.

Recipe (stands in for the paper's trained Nanochat checkpoints and validation prompts, which are
not available offline): every matrix, including the embedding and the lm head, is N(0, 0.02); the
two output projections (attention out-proj, MLP down-proj) are additionally scaled by 1/sqrt(2L).
For n_streams > 1 each block has two n x n residual-mixing matrices obtained by 20 Sinkhorn
iterations (row normalise, then column normalise) of exp(Z), Z ~ N(0, 1); the 1 x n pre-maps are
softmax(N(0,1)) and the n x 1 post-maps are 2*sigmoid(N(0,1)).  Token ids are uniform over the
vocabulary.
"""
from __future__ import annotations

from dataclasses import dataclass, asdict
from types import SimpleNamespace

import numpy as np


@dataclass
class ModelConfig:
    n_layer: int = 4
    d_model: int = 64
    n_head: int = 2
    head_dim: int = 32
    d_ff: int = 256
    vocab: int = 256
    n_streams: int = 1
    dtype: str = "fp32"  # "fp32" or "bf16": operand type of weights / GEMM inputs / KV cache
    rms_eps: float = 1e-6
    rope_base: float = 10000.0

    def as_dict(self):
        return asdict(self)


# The five workload shapes (random-init Nanochat-shaped models).
CONFIGS = {
    "tiny": ModelConfig(4, 64, 2, 32, 256, 256, 1, "fp32"),
    "d12": ModelConfig(12, 768, 6, 128, 3072, 32768, 1, "bf16"),
    "d20": ModelConfig(20, 1280, 10, 128, 5120, 65536, 1, "bf16"),
    "d20_hc": ModelConfig(20, 1280, 10, 128, 5120, 65536, 4, "bf16"),
    # the shape of the paper's own 0.5B model without x0-residual / value embeddings (Sec. 5: 32 layers, n_embd 640,
    # 5 heads); MLP width 4 d and the 65536-entry vocabulary are the Nanochat defaults, not stated in the paper
    "paper_0p5b": ModelConfig(32, 640, 5, 128, 2560, 65536, 1, "bf16"),
}


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even); result stays float32."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = ((u >> 16) & 1) + np.uint32(0x7FFF)
    u2 = ((u + r) & np.uint32(0xFFFF0000)).astype(np.uint32)
    return u2.view(np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """Upper 16 bits of float32 values that are already bf16-representable."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    return (u >> 16).astype(np.uint16)


def sinkhorn(logits: np.ndarray, iters: int = 20) -> np.ndarray:
    m = np.exp(logits.astype(np.float64))
    for _ in range(iters):
        m = m / m.sum(axis=-1, keepdims=True)
        m = m / m.sum(axis=-2, keepdims=True)
    return m


def make_weights(cfg: ModelConfig, seed: int = 1234, mix_seed: int = 5, std: float = 0.02,
                 embed_std: float | None = None) -> SimpleNamespace:
    """Random-init weights as float32 numpy arrays (bf16-representable when cfg.dtype == 'bf16')."""
    L, d, ff, V, n = cfg.n_layer, cfg.d_model, cfg.d_ff, cfg.vocab, cfg.n_streams
    assert cfg.n_head * cfg.head_dim == d
    rng = np.random.Generator(np.random.Philox(seed))

    def normal(shape, s):
        w = rng.standard_normal(shape, dtype=np.float32) * np.float32(s)
        return round_to_bf16(w) if cfg.dtype == "bf16" else w

    out_scale = 1.0 / np.sqrt(2.0 * L)
    W = SimpleNamespace()
    W.embed = normal((V, d), std if embed_std is None else embed_std)
    W.lm_head = normal((V, d), std)
    W.wqkv = normal((L, 3 * d, d), std)          # rows [0,d) = Wq, [d,2d) = Wk, [2d,3d) = Wv
    W.wo = normal((L, d, d), std * out_scale)
    W.wup = normal((L, ff, d), std)
    W.wdn = normal((L, d, ff), std * out_scale)
    _add_mixing(W, cfg, mix_seed)
    return W


def _add_mixing(W: SimpleNamespace, cfg: ModelConfig, mix_seed: int) -> None:
    """The stream-mixing maps of an n-stream model (their own generator: they do not depend on the dense weights)."""
    L, n = cfg.n_layer, cfg.n_streams
    if n > 1:
        mrng = np.random.Generator(np.random.Philox(mix_seed))
        W.hc_res_attn = sinkhorn(mrng.standard_normal((L, n, n))).astype(np.float32)
        W.hc_res_mlp = sinkhorn(mrng.standard_normal((L, n, n))).astype(np.float32)

        def softmax(z):
            e = np.exp(z - z.max(axis=-1, keepdims=True))
            return e / e.sum(axis=-1, keepdims=True)

        W.hc_pre_attn = softmax(mrng.standard_normal((L, n))).astype(np.float32)
        W.hc_pre_mlp = softmax(mrng.standard_normal((L, n))).astype(np.float32)
        W.hc_post_attn = (2.0 / (1.0 + np.exp(-mrng.standard_normal((L, n))))).astype(np.float32)
        W.hc_post_mlp = (2.0 / (1.0 + np.exp(-mrng.standard_normal((L, n))))).astype(np.float32)
    else:
        W.hc_res_attn = W.hc_res_mlp = None
        W.hc_pre_attn = W.hc_pre_mlp = W.hc_post_attn = W.hc_post_mlp = None


def with_mixing(W: SimpleNamespace, cfg: ModelConfig, mix_seed: int = 5) -> SimpleNamespace:
    """The weights make_weights(cfg, same seed, mix_seed) would return, built from an already generated set `W` of a
    model with the same dense shapes (the dense arrays are shared, not copied; only the mixing maps are drawn)."""
    out = SimpleNamespace(**{k: getattr(W, k) for k in ("embed", "lm_head", "wqkv", "wo", "wup", "wdn")})
    _add_mixing(out, cfg, mix_seed)
    return out


def with_embed_std(W: SimpleNamespace, cfg: ModelConfig, seed: int, embed_std: float) -> SimpleNamespace:
    """The weights make_weights(cfg, seed, embed_std=embed_std) would return, built from `W` = make_weights(cfg, seed):
    the embedding is the generator's first draw, so only it is drawn again, at the new scale."""
    rng = np.random.Generator(np.random.Philox(seed))
    e = rng.standard_normal((cfg.vocab, cfg.d_model), dtype=np.float32) * np.float32(embed_std)
    out = SimpleNamespace(**vars(W))
    out.embed = round_to_bf16(e) if cfg.dtype == "bf16" else e
    return out


def make_ids(cfg: ModelConfig, B: int, T: int, seed: int = 1) -> np.ndarray:
    rng = np.random.Generator(np.random.Philox(seed))
    return rng.integers(0, cfg.vocab, size=(B, T), dtype=np.int32)


def make_hidden(cfg: ModelConfig, B: int, T: int, seed: int = 7, std: float = 1.0) -> np.ndarray:
    """A random hidden state [B, T, n, d] (float32) for tests that bypass the embedding."""
    rng = np.random.Generator(np.random.Philox(seed))
    return (rng.standard_normal((B, T, cfg.n_streams, cfg.d_model), dtype=np.float32) * np.float32(std))
