"""Syntax-enriched training labels (Sec. III-C). TEST INFRASTRUCTURE ONLY.

L_0 is the token sequence with [FRAG] markers; head i's label row is L_0 shifted left by i
and padded with [PAD] to the same length; the rows are stacked into Labels of shape
(num_heads + 1, sequence_length). For each sequence position (column) the last [FRAG] along
the head axis is found and every label beyond it is replaced by [IGNORE]. A column with no
[FRAG] at all keeps only the base model's label (row 0): the paper does not say, this is the
reading taken. Plain loops over a matrix that is built exactly as the text describes.
"""
import numpy as np


def shifted_rows(l0, num_heads: int, pad: int) -> np.ndarray:
    l0 = np.asarray(l0, dtype=np.int64)
    n = len(l0)
    labels = np.full((num_heads + 1, n), pad, dtype=np.int64)
    for i in range(num_heads + 1):
        row = l0[i:]                       # L_i = L_0[i:]
        labels[i, :len(row)] = row         # [PAD] fills the rest
    return labels


def syntax_enriched_labels(l0, num_heads: int, frag: int, pad: int, ignore: int) -> np.ndarray:
    labels = shifted_rows(l0, num_heads, pad)
    for s in range(labels.shape[1]):
        last = 0
        for i in range(num_heads + 1):
            if labels[i, s] == frag:
                last = i
        for i in range(last + 1, num_heads + 1):
            labels[i, s] = ignore
    return labels
