"""Streams the seeded synthetic weights to a torch device tensor by tensor (so that a 7B
shape never needs all float32 draws in host memory at once). Produces the dictionary layout
the CUDA binding expects: q, k and v of a layer in one allocation ("wqkv"), gains float32,
everything else in the configuration's operand type. Input plumbing only."""
from concurrent.futures import ThreadPoolExecutor
from typing import Dict

import numpy as np

from .configs import ModelConfig
from .weights import draw_tensor, tensor_specs


def stream_weights_to_device(cfg: ModelConfig, device="cuda:0", threads: int = 8, keep_host=None) -> Dict[str, object]:
    """keep_host: optional dict that receives the float32 numpy draws (for the CPU oracle)."""
    import torch
    dt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    specs = tensor_specs(cfg)
    out: Dict[str, object] = {}
    qkv_rows = (cfg.n_heads + 2 * cfg.n_kv_heads) * cfg.head_dim
    qrows, krows = cfg.n_heads * cfg.head_dim, cfg.n_kv_heads * cfg.head_dim
    for l in range(cfg.n_layers):
        out[f"layers.{l}.wqkv"] = torch.empty((qkv_rows, cfg.d_model), dtype=dt, device=device)

    def job(item):
        idx, (name, shape, kind) = item
        return name, kind, draw_tensor(cfg, idx, shape, kind)

    with ThreadPoolExecutor(max_workers=max(1, threads)) as ex:
        window = 2 * max(1, threads)
        items = list(enumerate(specs))
        pending = []
        pos = 0
        while pos < len(items) or pending:
            while pos < len(items) and len(pending) < window:
                pending.append(ex.submit(job, items[pos]))
                pos += 1
            name, kind, arr = pending.pop(0).result()
            if keep_host is not None:
                keep_host[name] = arr
            t = torch.from_numpy(arr).to(device)
            t = t.to(torch.float32 if kind == "gain" else dt)
            leaf = name.split(".")[-1]
            if leaf in ("wq", "wk", "wv"):
                l = int(name.split(".")[1])
                r0 = {"wq": 0, "wk": qrows, "wv": qrows + krows}[leaf]
                out[f"layers.{l}.wqkv"][r0:r0 + t.shape[0]].copy_(t)
            else:
                out[name] = t.contiguous()
            del t
    return out
