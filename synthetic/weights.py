"""Seeded synthetic weights: every matrix, the embedding, lm_head, head matrices and
head biases are N(0, 0.02) draws in float32; RMSNorm gains are 1.0 (or 1 + 0.1 N(0,1)
when the config asks for random gains, which tests use so that a dropped gain shows).

Tensor t of the fixed order below is drawn from
numpy.random.default_rng(SeedSequence([seed, t])). Linear weights are row-major
[out_features, in_features]. Rounding to bf16 is left to the consumer.
"""
from concurrent.futures import ThreadPoolExecutor
from typing import Dict, List, Tuple

import numpy as np

from .configs import ModelConfig

LAYER_TENSORS = ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")


def tensor_specs(cfg: ModelConfig) -> List[Tuple[str, Tuple[int, ...], str]]:
    """(name, shape, kind) in the fixed draw order; kind is "normal" or "gain"."""
    d, hd = cfg.d_model, cfg.head_dim
    specs = [("embed", (cfg.vocab, d), "normal"),
             ("lm_head", (cfg.vocab, d), "normal"),
             ("final_norm", (d,), "gain")]
    for l in range(cfg.n_layers):
        shapes = {"attn_norm": (d,), "wq": (cfg.n_heads * hd, d), "wk": (cfg.n_kv_heads * hd, d),
                  "wv": (cfg.n_kv_heads * hd, d), "wo": (d, cfg.n_heads * hd), "ffn_norm": (d,),
                  "w_gate": (cfg.d_ffn, d), "w_up": (cfg.d_ffn, d), "w_down": (d, cfg.d_ffn)}
        for nm in LAYER_TENSORS:
            specs.append((f"layers.{l}.{nm}", shapes[nm], "gain" if nm.endswith("norm") else "normal"))
    for k in range(cfg.n_medusa):
        specs.append((f"medusa.{k}.w", (d, d), "normal"))
        specs.append((f"medusa.{k}.b", (d,), "normal"))
    return specs


def draw_tensor(cfg: ModelConfig, index: int, shape, kind: str) -> np.ndarray:
    rng = np.random.default_rng(np.random.SeedSequence([cfg.seed, index]))
    if kind == "gain":
        if cfg.norm_gain == "ones":
            return np.ones(shape, dtype=np.float32)
        return (1.0 + 0.1 * rng.standard_normal(shape, dtype=np.float32)).astype(np.float32)
    out = rng.standard_normal(shape, dtype=np.float32)
    out *= np.float32(0.02)
    return out


def draw_weights(cfg: ModelConfig, threads: int = 8) -> Dict[str, np.ndarray]:
    """All tensors as float32 numpy arrays keyed by name (drawn in parallel per tensor)."""
    specs = tensor_specs(cfg)
    with ThreadPoolExecutor(max_workers=max(1, threads)) as ex:
        arrays = list(ex.map(lambda it: draw_tensor(cfg, it[0], it[1][1], it[1][2]), enumerate(specs)))
    return {spec[0]: arr for spec, arr in zip(specs, arrays)}
