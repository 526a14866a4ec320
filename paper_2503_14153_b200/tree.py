"""Fixed candidate tree of the draft step (Sec. III-B: the candidates are the top-k
predictions of the base model and of each extra head).

A candidate is a path (c_1..c_m): candidate rank c_j of head j at depth j, with c_j below
the per-head cap. Paths are ranked by cost = sum_j (c_j + 1), shorter paths first at equal
cost, then lexicographically; the tree is the root plus the n_nodes-1 cheapest paths.
Generated cost level by cost level, so that no full enumeration is needed.
"""
from typing import Dict, List, Sequence, Tuple

import numpy as np


def build_tree(caps: Sequence[int], n_nodes: int) -> Dict[str, np.ndarray]:
    caps = [int(c) for c in caps]
    K = len(caps)

    def compose(pos: int, length: int, cost: int):
        # ranks for heads pos..length-1 with (rank+1) summing to cost, lexicographic
        if pos == length:
            if cost == 0:
                yield ()
            return
        remaining = length - pos - 1
        for r in range(min(caps[pos], cost - remaining)):
            for rest in compose(pos + 1, length, cost - (r + 1)):
                yield (r,) + rest

    nodes: List[Tuple[int, ...]] = [()]
    max_cost = sum(caps)
    cost = 1
    while len(nodes) < n_nodes and cost <= max_cost:
        for length in range(1, K + 1):
            for p in compose(0, length, cost):
                if len(nodes) < n_nodes:
                    nodes.append(p)
        cost += 1
    if len(nodes) < n_nodes:
        raise ValueError("n_nodes exceeds the number of candidate paths")
    where = {p: i for i, p in enumerate(nodes)}
    parent = np.array([-1] + [where[p[:-1]] for p in nodes[1:]], dtype=np.int32)
    depth = np.array([len(p) for p in nodes], dtype=np.int32)
    rank = np.array([0] + [p[-1] for p in nodes[1:]], dtype=np.int32)
    return {"parent": parent, "depth": depth, "rank": rank}


def chain_tree(length: int) -> Dict[str, np.ndarray]:
    """Root plus the rank-0 candidate of each successive head."""
    return {"parent": np.arange(-1, length - 1, dtype=np.int32),
            "depth": np.arange(length, dtype=np.int32),
            "rank": np.zeros(length, dtype=np.int32)}
