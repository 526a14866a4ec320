"""Acceptance rules of the verify step. TEST INFRASTRUCTURE ONLY.

Sec. III-B: a candidate token is accepted only if the rule holds for it and for all
tokens before it; the step's output is the longest accepted prefix among all candidates.
Greedy rule (the lossless mode): a node is accepted iff its token equals the base model's
argmax at its parent. Typical rule: Eq. 1.
"""
import numpy as np


def argmax_lowest(logits_f32: np.ndarray) -> np.ndarray:
    """Row-wise argmax on float32 values, lowest index on ties."""
    return np.argmax(np.asarray(logits_f32, dtype=np.float32), axis=-1).astype(np.int32)


def select_path(parent, depth, accepted_edge) -> list:
    """Longest prefix-closed accepted path; lowest node index among equally deep ones."""
    T = len(parent)
    acc = np.zeros(T, dtype=bool)
    acc[0] = True
    for v in range(1, T):
        acc[v] = acc[parent[v]] and bool(accepted_edge[v])
    best = 0
    for v in range(T):
        if acc[v] and depth[v] > depth[best]:
            best = v
    path = []
    v = best
    while v >= 0:
        path.append(v)
        v = int(parent[v])
    return path[::-1]


def greedy_accept(parent, depth, tok, am) -> list:
    """Node v != root passes iff tok[v] == am[parent[v]]."""
    T = len(parent)
    edge = np.zeros(T, dtype=bool)
    for v in range(1, T):
        edge[v] = tok[v] == am[parent[v]]
    return select_path(parent, depth, edge)


def typical_threshold(probs: np.ndarray, eps: float, delta: float) -> float:
    """Right-hand side of Eq. 1: min(eps, delta * exp(-H(p))), H in nats."""
    p = probs[probs > 0]
    H = float(-(p * np.log(p)).sum())
    return min(eps, delta * np.exp(-H))


def typical_accept(parent, depth, tok, logits, eps: float, delta: float, temperature: float = 1.0) -> list:
    """Node v != root passes iff p_base(tok[v] | prefix ending at parent) exceeds the
    threshold of Eq. 1 computed from the same distribution."""
    T = len(parent)
    edge = np.zeros(T, dtype=bool)
    cache = {}
    for v in range(1, T):
        u = int(parent[v])
        if u not in cache:
            z = np.asarray(logits[u], dtype=np.float64) / temperature
            z = z - z.max()
            p = np.exp(z)
            p /= p.sum()
            cache[u] = (p, typical_threshold(p, eps, delta))
        p, thr = cache[u]
        edge[v] = p[tok[v]] > thr
    return select_path(parent, depth, edge)


def sample_token(logits, temperature: float, u: float) -> int:
    """Sampled decoding at a temperature: the token drawn from softmax(logits / temperature) by
    inverting the cumulative distribution in token order at the uniform u in [0, 1): the first
    token j whose cumulative weight sum_{i <= j} exp((z_i - max z) / temperature) exceeds
    u times the total weight."""
    z = np.asarray(logits, dtype=np.float64) / temperature
    w = np.exp(z - z.max())
    cdf = np.cumsum(w)
    j = int(np.searchsorted(cdf, u * cdf[-1], side="right"))
    return min(j, len(w) - 1)


def truncate_to_fragment(path_tokens, frag_token: int) -> int:
    """Fragment-integrity rule of Sec. III-B: keep the accepted span up to and including
    its last fragment marker; with no marker in the span only the first token is kept.
    Returns the number of tokens kept (>= 1)."""
    keep = 1
    for i, t in enumerate(path_tokens):
        if t == frag_token:
            keep = i + 1
    return keep
