"""Llama-style decoder forward, extra decoding heads and top-k. TEST INFRASTRUCTURE ONLY.

Follows Sec. III-B: the base model scores every candidate position
(p_base(x_{t+i+1} | x_1..x_{t+i}) in Eq. 1) and the extra heads sit on the last hidden
state. float64 arithmetic; for "bf16" models operands are quantised at the fixed points
named in oracle.numerics.
"""
from concurrent.futures import ThreadPoolExecutor
from typing import Dict

import numpy as np

from .numerics import make_quantiser, round_bf16, silu


class OracleModel:
    """Holds the weights (float32 arrays keyed as in synthetic.weights) and the shape."""

    def __init__(self, cfg, weights: Dict[str, np.ndarray]):
        self.cfg = cfg
        self.q = make_quantiser(cfg.dtype)
        if cfg.dtype == "bf16":
            # weights are bf16 values: round every matrix and head bias once (per tensor, in threads)
            names = [k for k, v in weights.items() if v.ndim == 2 or ".b" in k]
            with ThreadPoolExecutor(max_workers=8) as ex:
                rounded = list(ex.map(lambda k: round_bf16(weights[k]).astype(np.float32), names))
            self.w = dict(weights)
            self.w.update(dict(zip(names, rounded)))
        else:
            self.w = dict(weights)

    def mat(self, name: str) -> np.ndarray:
        return self.w[name].astype(np.float64)


def rms_norm(x: np.ndarray, gain: np.ndarray, eps: float) -> np.ndarray:
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * gain


def rope_angles(positions: np.ndarray, head_dim: int, base: float):
    """cos/sin of pos * base^(-2i/D) for i in [0, D/2), float64."""
    i = np.arange(head_dim // 2, dtype=np.float64)
    inv_freq = base ** (-2.0 * i / head_dim)
    ang = np.asarray(positions, dtype=np.float64)[:, None] * inv_freq[None, :]
    return np.cos(ang), np.sin(ang)


def apply_rope(x: np.ndarray, cos: np.ndarray, sin: np.ndarray) -> np.ndarray:
    """x[T, H, D]; element i pairs with i + D/2 (rotate-half convention)."""
    half = x.shape[-1] // 2
    x1, x2 = x[..., :half], x[..., half:]
    c, s = cos[:, None, :], sin[:, None, :]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def masked_attention(q, k, v, vis, quant) -> np.ndarray:
    """q[T,H,D], k/v[S,Hkv,D], vis[T,S] bool -> [T,H,D]. Scale 1/sqrt(D); query head h
    reads KV head h // (H / Hkv). Probabilities are quantised before the value product."""
    T, H, D = q.shape
    Hkv = k.shape[1]
    group = H // Hkv
    out = np.empty((T, H, D), dtype=np.float64)
    scale = 1.0 / np.sqrt(D)
    for h in range(H):
        kh, vh = k[:, h // group, :], v[:, h // group, :]
        s = (q[:, h, :] @ kh.T) * scale
        s = np.where(vis, s, -np.inf)
        s = s - s.max(axis=-1, keepdims=True)
        e = np.exp(s)
        denom = e.sum(axis=-1, keepdims=True)
        out[:, h, :] = (quant(e) @ vh) / denom
    return out


class KVCache:
    """Logical cache: K and V rows per layer at slots 0..max_seq-1 (float64 values)."""

    def __init__(self, cfg, max_seq: int):
        shape = (cfg.n_layers, max_seq, cfg.n_kv_heads, cfg.head_dim)
        self.k = np.zeros(shape, dtype=np.float64)
        self.v = np.zeros(shape, dtype=np.float64)


def forward_rows(model: OracleModel, cache: KVCache, n: int, tok, pos, vis_rows, want_logits_rows=None):
    """Run the decoder on T new rows on top of n cached positions.

    tok[T], pos[T]: token ids and RoPE positions of the rows; vis_rows[T,T]: which new
    rows each row sees (all n cached positions are visible to every row). The rows' K/V
    are written to cache slots n..n+T-1. Returns (hidden[T,d] after the final norm,
    logits[rows,V] as float64 of the float32 logits).
    """
    cfg, q = model.cfg, model.q
    T = len(tok)
    H, Hkv, D = cfg.n_heads, cfg.n_kv_heads, cfg.head_dim
    x = model.mat("embed")[np.asarray(tok)]
    cos, sin = rope_angles(pos, D, cfg.rope_base)
    cos, sin = cos.astype(np.float32).astype(np.float64), sin.astype(np.float32).astype(np.float64)
    vis = np.concatenate([np.ones((T, n), dtype=bool), np.asarray(vis_rows, dtype=bool)], axis=1)
    for l in range(cfg.n_layers):
        p = f"layers.{l}."
        u = q(rms_norm(x, model.mat(p + "attn_norm"), cfg.rms_eps))
        qh = (u @ model.mat(p + "wq").T).reshape(T, H, D)
        kh = (u @ model.mat(p + "wk").T).reshape(T, Hkv, D)
        vh = (u @ model.mat(p + "wv").T).reshape(T, Hkv, D)
        qh, kh, vh = q(apply_rope(qh, cos, sin)), q(apply_rope(kh, cos, sin)), q(vh)
        cache.k[l, n:n + T] = kh
        cache.v[l, n:n + T] = vh
        o = masked_attention(qh, cache.k[l, :n + T], cache.v[l, :n + T], vis, q)
        x = x + q(o.reshape(T, H * D)) @ model.mat(p + "wo").T
        u = q(rms_norm(x, model.mat(p + "ffn_norm"), cfg.rms_eps))
        g = u @ model.mat(p + "w_gate").T
        up = u @ model.mat(p + "w_up").T
        x = x + q(silu(g) * up) @ model.mat(p + "w_down").T
    hidden = rms_norm(x, model.mat("final_norm"), cfg.rms_eps)
    rows = np.arange(T) if want_logits_rows is None else np.asarray(want_logits_rows)
    logits = q(hidden[rows]) @ model.mat("lm_head").T
    return hidden, logits.astype(np.float32).astype(np.float64)


def forward_full(model: OracleModel, tokens) -> np.ndarray:
    """No-cache definition: causal forward over the whole sequence, logits of every row."""
    n = len(tokens)
    cache = KVCache(model.cfg, n)
    vis = np.tril(np.ones((n, n), dtype=bool))
    _, logits = forward_rows(model, cache, 0, tokens, np.arange(n), vis)
    return logits


def medusa_logits(model: OracleModel, hidden_last: np.ndarray) -> np.ndarray:
    """z_k = W_lm (h + SiLU(W_k h + b_k)) for each extra head k (shared lm_head); [K,V]."""
    cfg, q = model.cfg, model.q
    h = q(hidden_last)
    out = np.empty((cfg.n_medusa, cfg.vocab), dtype=np.float64)
    for k in range(cfg.n_medusa):
        r = h + silu(model.mat(f"medusa.{k}.w") @ h + model.mat(f"medusa.{k}.b"))
        out[k] = model.mat("lm_head") @ q(r)
    return out.astype(np.float32).astype(np.float64)


def top_k(values_f32: np.ndarray, k: int) -> np.ndarray:
    """Indices of the k largest values, by (value descending, index ascending)."""
    v = np.asarray(values_f32, dtype=np.float32)
    order = np.lexsort((np.arange(len(v)), -v.astype(np.float64)))
    return order[:k].astype(np.int32)
