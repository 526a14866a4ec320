"""How far the bf16 rounding contract itself moves a result when only the accumulation precision
changes. TEST INFRASTRUCTURE ONLY.

The oracle rounds operands to bf16 at fixed points and accumulates in float64; a tensor-core
implementation of the same contract accumulates in float32. Wherever the two sums fall on
different sides of a bf16 rounding boundary, one operand element differs by one unit in the last
place, and later layers amplify it. This script runs the oracle's own forward twice on the same
seeded weights and prompt -- float64 accumulation, and float32 matrices, activations and
products (OracleModelF32) -- at several depths and prints max|a-b| / max|b| of the last hidden
rows, of the logits rows, and the largest top-2 logit gap at which the two runs pick different
argmax tokens. It says how tight a tolerance any float32-accumulating implementation can be held
to at that depth; it involves no GPU code.

    python -m oracle.sensitivity --config c1 --depths 1 2 4 8 16 32 --rows 16
"""
import argparse
import time

import numpy as np

from .decoder import KVCache, OracleModel, forward_rows
from .numerics import round_bf16


class OracleModelF32(OracleModel):
    """Same weights and rounding points; matrices and activations stay float32, so every
    projection is a float32 product with float32 accumulation."""

    def __init__(self, cfg, weights):
        super().__init__(cfg, weights)
        self.q = lambda x: round_bf16(x).astype(np.float32)

    def mat(self, name):
        return self.w[name]


def depth_sensitivity(cfg, weights, depths, prompt, rows):
    """For each depth L (the first L layers of `weights`): the two runs over a causal chain of
    `rows` tokens after nothing cached. Returns a list of dicts."""
    out = []
    tok = np.asarray(prompt[:rows])
    vis = np.tril(np.ones((rows, rows), dtype=bool))
    for L in depths:
        c = cfg.with_(n_layers=L)
        res = []
        for cls in (OracleModel, OracleModelF32):
            m = cls(c, weights)
            t0 = time.time()
            hid, lg = forward_rows(m, KVCache(c, rows), 0, tok, np.arange(rows), vis)
            res.append((np.asarray(hid, np.float64), np.asarray(lg, np.float64), time.time() - t0))
            del m
        (h0, l0, t_a), (h1, l1, t_b) = res
        rel = lambda a, b: float(np.max(np.abs(a - b).max(axis=1) / np.abs(b).max(axis=1)))
        a0, a1 = l0.argmax(axis=1), l1.argmax(axis=1)
        flips = np.nonzero(a0 != a1)[0]
        gaps = [float(l0[r, a0[r]] - l0[r, a1[r]]) for r in flips]
        srt = np.sort(l0, axis=1)
        out.append({"layers": L, "hidden": rel(h1, h0), "logits": rel(l1, l0), "argmax_flips": len(flips),
                    "largest_flip_gap": max(gaps) if gaps else 0.0, "rows": rows,
                    "median_top2_gap": float(np.median(srt[:, -1] - srt[:, -2])), "max_abs_logit": float(np.abs(l0).max()),
                    "seconds": (round(t_a, 1), round(t_b, 1))})
        print(out[-1], flush=True)
    return out


def main():
    from synthetic import draw_prompt, draw_tensor, get_config, tensor_specs
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="c1")
    ap.add_argument("--depths", type=int, nargs="+", default=[1, 2, 4, 8, 16, 32])
    ap.add_argument("--rows", type=int, default=16)
    args = ap.parse_args()
    cfg = get_config(args.config)
    top = max(args.depths)
    w = {}
    for idx, (name, shape, kind) in enumerate(tensor_specs(cfg)):
        if name.startswith("layers.") and int(name.split(".")[1]) >= top:
            continue
        if name.startswith("medusa."):
            continue
        w[name] = draw_tensor(cfg, idx, shape, kind)
    depth_sensitivity(cfg, w, args.depths, draw_prompt(cfg, args.rows), args.rows)


if __name__ == "__main__":
    main()
