"""Seeded prompts and the controlled-acceptance draft table.

Prompts are uniform random token ids; they stand in for the paper's evaluation prompts
(Sec. IV-B), which are not reproduced here.
"""
from typing import List

import numpy as np

from .configs import ModelConfig


def draw_prompt(cfg: ModelConfig, length: int = None) -> np.ndarray:
    rng = np.random.default_rng(np.random.SeedSequence([cfg.seed, 10_000]))
    n = cfg.prompt_len if length is None else length
    return rng.integers(0, cfg.vocab, size=n, dtype=np.int64).astype(np.int32)


def draw_prompt_batch(cfg: ModelConfig, batch: int, lo: int, hi: int) -> List[np.ndarray]:
    """`batch` prompts with lengths i.i.d. uniform integers in [lo, hi]."""
    rng = np.random.default_rng(np.random.SeedSequence([cfg.seed, 10_001]))
    lens = rng.integers(lo, hi + 1, size=batch)
    return [rng.integers(0, cfg.vocab, size=int(n), dtype=np.int64).astype(np.int32) for n in lens]


def controlled_draft(cfg: ModelConfig, greedy_stream: np.ndarray, p: float, n_steps: int) -> np.ndarray:
    """Per-step candidate tables for the controlled-acceptance draft.

    greedy_stream[i] is the base model's greedy token at generated position i (position 0
    is the first root token). Returns uniforms[n_steps, K, kmax] int32 and a Bernoulli
    table hit[n_steps, K]; the harness, which knows how many tokens are committed at a
    step, writes greedy_stream[done + j] into rank 0 of head j where hit is set.
    """
    rng = np.random.default_rng(np.random.SeedSequence([cfg.seed, 20_000, int(round(p * 1000))]))
    uniforms = rng.integers(0, cfg.vocab, size=(n_steps, cfg.n_medusa, cfg.kmax), dtype=np.int64).astype(np.int32)
    hit = rng.random(size=(n_steps, cfg.n_medusa)) < p
    return uniforms, hit
