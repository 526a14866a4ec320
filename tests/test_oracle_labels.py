"""Pins of the oracle's syntax-enriched label construction (Sec. III-C)."""
import os

import numpy as np

from oracle.labels import shifted_rows, syntax_enriched_labels

HERE = os.path.dirname(os.path.abspath(__file__))
FRAG, PAD, IGN = 9, 0, -100


def test_worked_example_by_hand():
    rows = {}
    for line in open(os.path.join(HERE, "golden", "labels_worked_example.txt")):
        if line.startswith("#") or not line.strip():
            continue
        k, *v = line.split()
        rows[k] = np.array([int(x) for x in v])
    got = syntax_enriched_labels(rows["l0"], 3, FRAG, PAD, IGN)
    want = np.stack([rows[f"row{i}"] for i in range(4)])
    assert np.array_equal(got, want)


def test_shape_shift_and_padding():
    rng = np.random.default_rng(0)
    l0 = rng.integers(1, 8, size=37)
    lab = shifted_rows(l0, 5, PAD)
    assert lab.shape == (6, 37)
    for i in range(6):
        assert np.array_equal(lab[i, :37 - i], l0[i:]) and np.all(lab[i, 37 - i:] == PAD)


def test_columns_end_on_a_marker_and_ignores_grow_with_the_head_index():
    rng = np.random.default_rng(1)
    l0 = rng.integers(1, 8, size=400)
    l0[rng.random(400) < 0.2] = FRAG
    K = 10
    lab = syntax_enriched_labels(l0, K, FRAG, PAD, IGN)
    assert np.array_equal(lab[0], l0)                     # the base model's labels are never touched
    raw = shifted_rows(l0, K, PAD)
    for s in range(400):
        kept = np.where(lab[:, s] != IGN)[0]
        assert np.array_equal(kept, np.arange(len(kept)))  # a prefix along the head axis is kept
        last = kept[-1]
        assert np.array_equal(lab[kept, s], raw[kept, s])  # kept labels are the shifted tokens
        assert last == 0 or lab[last, s] == FRAG           # the kept fragment ends on a marker
        assert not np.any(raw[last + 1:, s] == FRAG)       # and no marker was thrown away
    frac = [(lab[i] == IGN).mean() for i in range(K + 1)]
    assert all(b >= a for a, b in zip(frac, frac[1:]))     # later heads ignore more (Sec. III-C)


def test_no_marker_and_all_markers():
    l0 = np.arange(1, 9)
    lab = syntax_enriched_labels(l0, 2, FRAG, PAD, IGN)
    assert np.array_equal(lab[0], l0) and np.all(lab[1:] == IGN)
    lab = syntax_enriched_labels(np.full(6, FRAG), 2, FRAG, PAD, IGN)
    want = shifted_rows(np.full(6, FRAG), 2, PAD)
    want[1, 5] = IGN; want[2, 4:] = IGN                    # beyond the row's end only [PAD] follows the last marker
    assert np.array_equal(lab, want)
