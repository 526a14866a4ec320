"""Candidate tree of the draft step. TEST INFRASTRUCTURE ONLY.

Sec. III-B keeps "several candidates" made of the top-k predictions of the base model and
of each head, and picks the longest accepted prefix among them. A candidate is a path
(c_1..c_m): rank c_j of head j at depth j. The fixed tree is the T-1 cheapest paths under
the key (sum_j (c_j+1), length, path), plus the root (the base model's own token).
"""
import itertools
from typing import Dict, List, Tuple

import numpy as np


def enumerate_paths(caps) -> List[Tuple[int, ...]]:
    paths = []
    for m in range(1, len(caps) + 1):
        for p in itertools.product(*[range(c) for c in caps[:m]]):
            paths.append(p)
    return paths


def build_tree(caps, n_nodes: int) -> Dict[str, np.ndarray]:
    paths = enumerate_paths(caps)
    paths.sort(key=lambda p: (sum(c + 1 for c in p), len(p), p))
    if n_nodes - 1 > len(paths):
        raise ValueError("tree larger than the number of candidate paths")
    chosen = [()] + paths[: n_nodes - 1]
    index = {p: i for i, p in enumerate(chosen)}
    parent = np.full(n_nodes, -1, dtype=np.int32)
    depth = np.zeros(n_nodes, dtype=np.int32)
    rank = np.zeros(n_nodes, dtype=np.int32)
    for i, p in enumerate(chosen):
        if i == 0:
            continue
        parent[i] = index[p[:-1]]
        depth[i] = len(p)
        rank[i] = p[-1]
    return {"parent": parent, "depth": depth, "rank": rank, "paths": chosen}


def chain_tree(length: int) -> Dict[str, np.ndarray]:
    """Root followed by rank-0 children only: node i's parent is i-1."""
    parent = np.arange(-1, length - 1, dtype=np.int32)
    depth = np.arange(length, dtype=np.int32)
    rank = np.zeros(length, dtype=np.int32)
    return {"parent": parent, "depth": depth, "rank": rank}


def ancestor_mask(parent: np.ndarray) -> np.ndarray:
    """vis[v, u] = True iff u is v or an ancestor of v (parents precede children)."""
    T = len(parent)
    vis = np.zeros((T, T), dtype=bool)
    for v in range(T):
        if parent[v] >= 0:
            vis[v] = vis[parent[v]]
        vis[v, v] = True
    return vis


def validate_tree(parent, depth, rank, n_heads: int, kmax: int) -> None:
    T = len(parent)
    if T < 1 or parent[0] != -1 or depth[0] != 0 or rank[0] != 0:
        raise ValueError("node 0 must be the root")
    seen = set()
    for v in range(1, T):
        p = int(parent[v])
        if not (0 <= p < v):
            raise ValueError("parent must precede child")
        if depth[v] != depth[p] + 1 or depth[v] > n_heads:
            raise ValueError("bad depth")
        if not (0 <= rank[v] < kmax):
            raise ValueError("bad rank")
        if (p, int(rank[v])) in seen:
            raise ValueError("siblings share a rank")
        seen.add((p, int(rank[v])))
