"""Lock-step draft-and-verify decoder and the plain greedy reference.
TEST INFRASTRUCTURE ONLY.

One step (Sec. III-B): the extra heads propose per-head top-k candidates from the last
accepted hidden state, the candidates fill the fixed tree, the base model scores every
tree node in one masked forward, the longest accepted prefix is emitted and its K/V rows
become the next cached positions.
"""
import numpy as np

from .accept import argmax_lowest, greedy_accept, sample_token, truncate_to_fragment, typical_accept
from .decoder import KVCache, OracleModel, forward_full, forward_rows, medusa_logits, top_k
from .rng import step_uniform
from .tree import ancestor_mask


def greedy_decode_nocache(model: OracleModel, prompt, new_tokens: int) -> np.ndarray:
    """Textbook greedy decoding, recomputing the whole forward for every token."""
    toks = list(int(t) for t in prompt)
    out = []
    for _ in range(new_tokens):
        logits = forward_full(model, toks)
        nxt = int(argmax_lowest(logits[-1]))
        out.append(nxt)
        toks.append(nxt)
    return np.asarray(out, dtype=np.int32)


class OracleSpecDecoder:
    def __init__(self, model: OracleModel, tree, max_seq: int, accept_mode: str = "greedy",
                 typ_eps: float = 0.09, typ_delta: float = 0.3, temperature: float = 1.0,
                 frag_token: int = -1, sampling: bool = False, seed: int = 0, sequence: int = 0):
        self.model, self.cfg = model, model.cfg
        self.parent = np.asarray(tree["parent"], dtype=np.int32)
        self.depth = np.asarray(tree["depth"], dtype=np.int32)
        self.rank = np.asarray(tree["rank"], dtype=np.int32)
        self.T = len(self.parent)
        self.vis = ancestor_mask(self.parent)
        self.cache = KVCache(self.cfg, max_seq + self.T)
        self.accept_mode = accept_mode
        self.typ = (typ_eps, typ_delta, temperature)
        self.frag_token = frag_token
        # sampled decoding (Sec. IV-B times every prompt greedy and at temperature 0.8): the token that
        # follows the accepted span is drawn from softmax(logits / temperature) instead of the argmax
        self.sampling, self.seed, self.sequence = sampling, seed, sequence
        self.draws = 0                      # draw counter: 0 for the token after the prompt, then one per step
        self.n = 0
        self.root_tok = None
        self.h_last = None

    # --- prefill: causal forward over the prompt; keeps last hidden and the first root ---
    def prefill(self, prompt, chunk: int = 128):
        prompt = np.asarray(prompt, dtype=np.int32)
        self.n = 0
        hidden = logits = None
        for s in range(0, len(prompt), chunk):
            part = prompt[s:s + chunk]
            c = len(part)
            hidden, logits = forward_rows(self.model, self.cache, self.n, part,
                                          np.arange(self.n, self.n + c),
                                          np.tril(np.ones((c, c), dtype=bool)), [c - 1])
            self.n += c
        self.h_last = hidden[-1]
        self.draws = 0
        self.root_tok = self._next_token(logits[0])
        self.last_root_logits = logits[0]

    def _next_token(self, logits_row) -> int:
        """Base model's own next token: the argmax, or in sampled decoding the draw at this step's uniform."""
        if not self.sampling:
            return int(argmax_lowest(logits_row))
        self.last_u = step_uniform(self.seed, self.sequence, self.draws)
        self.draws += 1
        return sample_token(logits_row, self.typ[2], self.last_u)

    def candidates(self):
        """cand[0][0] = root token; cand[k][j] = j-th best token of head k."""
        cfg = self.cfg
        z = medusa_logits(self.model, self.h_last)
        cand = np.full((cfg.n_medusa + 1, cfg.kmax), -1, dtype=np.int32)
        cand[0, 0] = self.root_tok
        for k in range(cfg.n_medusa):
            cand[k + 1, :cfg.topk[k]] = top_k(z[k], cfg.topk[k])
        return cand, z

    def step(self, cand_override=None):
        cand, z = self.candidates()
        if cand_override is not None:
            ov = np.asarray(cand_override, dtype=np.int32)
            keep = ov < 0
            cand[1:] = np.where(keep, cand[1:], ov)
        tok = cand[self.depth, self.rank]
        pos = self.n + self.depth
        hidden, logits = forward_rows(self.model, self.cache, self.n, tok, pos, self.vis)
        am = argmax_lowest(logits)
        if self.accept_mode == "greedy":
            path = greedy_accept(self.parent, self.depth, tok, am)
        else:
            path = typical_accept(self.parent, self.depth, tok, logits, *self.typ)
        if self.frag_token >= 0:
            path = path[:truncate_to_fragment([int(tok[v]) for v in path], self.frag_token)]
        count = len(path)
        for l in range(self.cfg.n_layers):
            self.cache.k[l, self.n:self.n + count] = self.cache.k[l, self.n + np.asarray(path)]
            self.cache.v[l, self.n:self.n + count] = self.cache.v[l, self.n + np.asarray(path)]
        best = path[-1]
        next_root = self._next_token(logits[best])
        rec = {"cand": cand, "head_logits": z, "tok": tok, "pos": pos, "logits": logits,
               "hidden": hidden, "am": am, "path": np.asarray(path, dtype=np.int32),
               "count": count, "tokens": tok[path].astype(np.int32), "n_before": self.n,
               "next_root": next_root, "best": int(best)}
        self.n += count
        self.root_tok = next_root
        self.h_last = hidden[best]
        return rec

    def force_commit(self, n_before: int, tokens, next_root: int):
        """Adopt another decoder's emitted tokens for the step that started at n_before:
        recompute their K/V rows and the last hidden as a chain, and take its next root."""
        tokens = np.asarray(tokens, dtype=np.int32)
        c = len(tokens)
        hidden, _ = forward_rows(self.model, self.cache, n_before, tokens,
                                 np.arange(n_before, n_before + c),
                                 np.tril(np.ones((c, c), dtype=bool)), [c - 1])
        self.n = n_before + c
        self.h_last = hidden[-1]
        self.root_tok = int(next_root)

    def generate(self, prompt, new_tokens: int, overrides=None):
        self.prefill(prompt)
        out, counts = [], []
        i = 0
        while len(out) < new_tokens:
            rec = self.step(None if overrides is None else overrides(i, len(out), self))
            out.extend(int(t) for t in rec["tokens"])
            counts.append(rec["count"])
            i += 1
        return np.asarray(out[:new_tokens], dtype=np.int32), counts
