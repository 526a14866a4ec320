"""Rounding helpers for the oracle. TEST INFRASTRUCTURE ONLY.

The bf16 configurations quantise operands at fixed points of the forward pass (normed
activations, q/k/v after RoPE, softmax probabilities, attention output, SiLU(g)*u, final
hidden, head block output); everything else stays in float64 here.
"""
import numpy as np


def round_bf16(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even to bfloat16 precision; returns float64 holding bf16 values."""
    f = np.ascontiguousarray(np.asarray(x, dtype=np.float32))
    u = f.view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    r = ((u + bias) & np.uint32(0xFFFF0000)).view(np.float32)
    nan = np.isnan(f)
    if nan.any():
        r = np.where(nan, f, r)
    return r.astype(np.float64)


def make_quantiser(dtype: str):
    """q(x): identity for "fp32"/"exact", bf16 rounding for "bf16"."""
    if dtype == "bf16":
        return round_bf16
    return lambda x: np.asarray(x, dtype=np.float64)


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))
