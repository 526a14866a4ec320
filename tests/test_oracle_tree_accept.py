"""Pins of the oracle's candidate tree, ancestor mask and acceptance rules."""
import itertools
import os

import numpy as np
import pytest

from oracle.accept import (greedy_accept, select_path, truncate_to_fragment, typical_accept,
                           typical_threshold)
from oracle.tree import ancestor_mask, build_tree, chain_tree, validate_tree

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "tree_depth_histograms.txt")


def _golden_rows():
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        left, right = line.split(":")
        caps, T = left.split()
        yield tuple(int(c) for c in caps.split(",")), int(T), [int(x) for x in right.split()]


@pytest.mark.parametrize("caps,T,hist", list(_golden_rows()))
def test_tree_depth_histogram(caps, T, hist):
    tree = build_tree(caps, T)
    assert list(np.bincount(tree["depth"])) == hist
    validate_tree(tree["parent"], tree["depth"], tree["rank"], len(caps), max(caps))


def test_tree_first_nodes_by_hand():
    # caps (4,2,2): order by cost then length then path
    tree = build_tree((4, 2, 2), 16)
    assert tree["paths"][:8] == [(), (0,), (1,), (0, 0), (2,), (0, 1), (1, 0), (0, 0, 0)]
    assert set(tree["paths"][14:]) == {(2, 1), (3, 0)}


@pytest.mark.parametrize("caps,T", [((4, 2, 2), 16), ((10, 4, 2, 2), 64), ((10, 4, 2, 2), 128), ((3, 3), 12)])
def test_tree_prefix_closed_distinct_and_contains_greedy_chain(caps, T):
    tree = build_tree(caps, T)
    paths = tree["paths"]
    assert len(set(paths)) == T
    for p in paths[1:]:
        assert p[:-1] in paths
        assert all(c < cap for c, cap in zip(p, caps))
    if T >= 16:
        for m in range(1, len(caps) + 1):
            assert tuple([0] * m) in paths


@pytest.mark.parametrize("caps,T", [((4, 2, 2), 16), ((10, 4, 2, 2), 64), ((10, 4, 2, 2), 128)])
def test_mask_equals_bruteforce_ancestors(caps, T):
    tree = build_tree(caps, T)
    parent, depth = tree["parent"], tree["depth"]
    vis = ancestor_mask(parent)
    brute = np.zeros((T, T), dtype=bool)
    for v in range(T):
        u = v
        while u != -1:
            brute[v, u] = True
            u = int(parent[u])
    assert np.array_equal(vis, brute)
    assert np.array_equal(vis, np.tril(vis))
    assert np.array_equal(vis.sum(axis=1), depth + 1)


def test_chain_mask_is_causal():
    assert np.array_equal(ancestor_mask(chain_tree(9)["parent"]), np.tril(np.ones((9, 9), bool)))


def test_validate_tree_rejects_bad_trees():
    t = build_tree((3, 2), 6)
    for mutate in (lambda p, d, r: p.__setitem__(0, 0),
                   lambda p, d, r: p.__setitem__(2, 4),
                   lambda p, d, r: d.__setitem__(3, 5),
                   lambda p, d, r: r.__setitem__(1, 9),
                   lambda p, d, r: r.__setitem__(2, int(r[1]))):
        p, d, r = t["parent"].copy(), t["depth"].copy(), t["rank"].copy()
        mutate(p, d, r)
        with pytest.raises(ValueError):
            validate_tree(p, d, r, 2, 3)


def _brute_longest(parent, depth, tok, am):
    """Try every root-to-node path; a path is accepted iff every non-root node on it
    carries the argmax token of its parent."""
    best_len, best_nodes = 1, [0]
    for v in range(len(parent)):
        nodes, u = [], v
        while u != -1:
            nodes.append(u); u = int(parent[u])
        nodes = nodes[::-1]
        ok = all(tok[c] == am[p] for p, c in zip(nodes[:-1], nodes[1:]))
        if ok and len(nodes) > best_len:
            best_len, best_nodes = len(nodes), nodes
    return best_len, best_nodes


def test_greedy_accept_equals_bruteforce_on_random_small_trees():
    rng = np.random.default_rng(0)
    for trial in range(300):
        caps = tuple(int(c) for c in rng.integers(1, 4, size=rng.integers(1, 5)))
        total = sum(int(np.prod(caps[:m])) for m in range(1, len(caps) + 1))
        T = int(rng.integers(1, min(total, 24) + 1)) + 1
        if T - 1 > total:
            T = total + 1
        tree = build_tree(caps, T)
        V = 3                                     # tiny vocabulary -> many matches
        tok = rng.integers(0, V, T)
        am = rng.integers(0, V, T)
        path = greedy_accept(tree["parent"], tree["depth"], tok, am)
        n, nodes = _brute_longest(tree["parent"], tree["depth"], tok, am)
        assert len(path) == n
        assert 1 <= len(path) <= len(caps) + 1
        assert path[0] == 0 and all(tree["parent"][c] == p for p, c in zip(path[:-1], path[1:]))
        assert all(tok[c] == am[p] for p, c in zip(path[:-1], path[1:]))
        if len(set(tok[1:])) == T - 1:            # distinct sibling tokens -> unique path
            assert path == nodes


def test_accept_tie_goes_to_lowest_node_index():
    # two depth-1 children both accepted (duplicate tokens): lowest index wins
    parent, depth = np.array([-1, 0, 0]), np.array([0, 1, 1])
    assert select_path(parent, depth, np.array([0, 1, 1], bool)) == [0, 1]
    assert select_path(parent, depth, np.array([0, 0, 1], bool)) == [0, 2]
    assert select_path(parent, depth, np.array([0, 0, 0], bool)) == [0]


def test_accept_is_prefix_closed():
    # child matches but its parent does not: nothing beyond the root is accepted
    parent, depth = np.array([-1, 0, 1]), np.array([0, 1, 2])
    assert greedy_accept(parent, depth, np.array([5, 6, 7]), np.array([9, 7, 0])) == [0]
    assert greedy_accept(parent, depth, np.array([5, 6, 7]), np.array([6, 7, 0])) == [0, 1, 2]


def test_typical_threshold_closed_forms():
    V = 50
    onehot = np.zeros(V); onehot[3] = 1.0
    assert typical_threshold(onehot, 0.09, 0.3) == pytest.approx(min(0.09, 0.3))       # H = 0
    assert typical_threshold(onehot, 0.5, 0.3) == pytest.approx(0.3)
    uni = np.full(V, 1.0 / V)
    assert typical_threshold(uni, 0.09, 0.3) == pytest.approx(min(0.09, 0.3 / V))      # exp(-ln V) = 1/V


def test_typical_accept_uniform_and_peaked():
    parent, depth = np.array([-1, 0, 1]), np.array([0, 1, 2])
    V = 10
    logits = np.zeros((3, V))                     # uniform: p = 0.1 > min(0.09, 0.03) -> all pass
    assert typical_accept(parent, depth, np.array([1, 2, 3]), logits, 0.09, 0.3) == [0, 1, 2]
    logits[0, 7] = 50.0                           # peaked at 7: token 2 has p ~ 0 -> stops at root
    assert typical_accept(parent, depth, np.array([1, 2, 3]), logits, 0.09, 0.3) == [0]
    assert typical_accept(parent, depth, np.array([1, 7, 3]), logits, 0.09, 0.3) == [0, 1, 2]


def test_fragment_truncation_rule():
    assert truncate_to_fragment([5, 9, 5, 4], 9) == 2
    assert truncate_to_fragment([5, 9, 5, 9], 9) == 4
    assert truncate_to_fragment([5, 6, 7], 9) == 1      # no marker: keep the root only
    assert truncate_to_fragment([9, 6, 7], 9) == 1


def test_typical_accept_temperature_two_token_closed_form():
    """Eq. 1 with p = softmax(logits / temperature) on a two-token vocabulary. Root logits
    (temperature * ln 3, 0) give p = (3/4, 1/4) at every temperature, H = ln 4 - (3/4) ln 3 and
    exp(-H) = 3^(3/4) / 4 = 0.56988; with eps = 1 the threshold is delta * 0.56988: 0.2849 at
    delta 0.5 and 0.2279 at delta 0.4. The child carries token 1 (p = 1/4), so it is rejected
    at delta 0.5 and accepted at delta 0.4, whatever the temperature. A rule that multiplied
    the logits by the temperature would see p = (0.568, 0.432) at temperature 0.5 (accepts at
    delta 0.5) and p = (81/82, 1/82) at temperature 2 (rejects at delta 0.4)."""
    assert 3 ** 0.75 / 4 == pytest.approx(0.5698768, abs=1e-6)
    parent, depth, tok = np.array([-1, 0]), np.array([0, 1]), np.array([0, 1])
    for temperature in (0.5, 1.0, 2.0):
        lg = np.zeros((2, 2))
        lg[0] = [temperature * np.log(3.0), 0.0]
        assert typical_accept(parent, depth, tok, lg, 1.0, 0.5, temperature) == [0]
        assert typical_accept(parent, depth, tok, lg, 1.0, 0.4, temperature) == [0, 1]
        # eps is the smaller bound: 0.2 < 0.2849 lets the p = 1/4 token through
        assert typical_accept(parent, depth, tok, lg, 0.2, 0.5, temperature) == [0, 1]
