"""Model shapes and run recipes of the five benchmark configurations.

Each entry fixes the decoder shape, the arithmetic type, the number of extra decoding
heads (Sec. III-B: head i predicts the token at t+i+1), the per-head top-k caps and the
candidate-tree size, the prompt length and the number of new tokens.
"""
from dataclasses import dataclass, replace
from typing import Tuple


@dataclass(frozen=True)
class ModelConfig:
    name: str
    n_layers: int
    d_model: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rms_eps: float
    rope_base: float
    dtype: str               # "fp32" or "bf16"
    n_medusa: int            # K extra heads
    topk: Tuple[int, ...]    # per-head top-k caps (k_1..k_K)
    tree_nodes: int          # T, root included
    prompt_len: int
    new_tokens: int
    seed: int
    page_size: int = 16
    batch: int = 1
    norm_gain: str = "ones"  # "ones" (benchmark recipe) or "random" (tests)

    def with_(self, **kw) -> "ModelConfig":
        return replace(self, **kw)

    @property
    def kmax(self) -> int:
        return max(self.topk) if self.topk else 1


_TINY = ModelConfig(
    name="c0_tiny_fp32", n_layers=2, d_model=256, n_heads=4, n_kv_heads=4, head_dim=64,
    d_ffn=688, vocab=32016, rms_eps=1e-5, rope_base=10000.0, dtype="fp32", n_medusa=3,
    topk=(4, 2, 2), tree_nodes=16, prompt_len=32, new_tokens=64, seed=0)

_7B = ModelConfig(
    name="c1_7b_bf16", n_layers=32, d_model=4096, n_heads=32, n_kv_heads=32, head_dim=128,
    d_ffn=11008, vocab=32016, rms_eps=1e-5, rope_base=1e6, dtype="bf16", n_medusa=4,
    topk=(10, 4, 2, 2), tree_nodes=64, prompt_len=256, new_tokens=256, seed=1)

CONFIGS = {
    "c0": _TINY,
    "c1": _7B,
    "c2": _7B.with_(name="c2_7b_controlled", prompt_len=512, new_tokens=512, seed=2),
    "c3": _7B.with_(name="c3_7b_long", prompt_len=8192, new_tokens=128, seed=3),
    "c4": _7B.with_(name="c4_7b_batch16", prompt_len=2048, new_tokens=256, seed=4, batch=16),
}


def get_config(key: str, **overrides) -> ModelConfig:
    cfg = CONFIGS[key]
    return cfg.with_(**overrides) if overrides else cfg
