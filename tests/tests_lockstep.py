"""Lock-step comparison of the CUDA decode loop with the CPU oracle (test harness).

Both decoders advance one step at a time from the same committed prefix. Token decisions
must agree exactly except at logged near ties, where the oracle adopts the CUDA path's decision
and the run continues. Logits and hidden states are compared per row with
max|a-b| / max|b| <= tol.

What counts as a near tie:
  * an argmax (or a head's top-k rank) may differ only where the oracle's gap between the two
    competing logits is below `tie_gap`; with `tie_from_row_error` the bound for a node is
    instead max(tie_gap, 2 x the largest absolute difference between the two sides' logits in
    that row), which is the most a row that close can move a decision (logged per case);
  * the emitted span or the next root may differ only if the last node the two accepted
    paths have in common is such a logged node (greedy rule), or, under Eq. 1, if a child of
    that node has its probability within `edge_tol` (relative) of the threshold;
  * a sampled next root may differ only if the oracle's u x total lies within `sample_tol` x
    total of the cumulative-weight interval of the token the CUDA path drew.
"""
from dataclasses import dataclass, field
from typing import Callable, Dict, List, Optional

import numpy as np

from oracle.accept import typical_threshold
from oracle.decoder import OracleModel
from oracle.spec import OracleSpecDecoder
from paper_2503_14153_b200 import SpecDecoder, upload_weights
from paper_2503_14153_b200 import binding as B


def rel_err_rows(a: np.ndarray, b: np.ndarray) -> float:
    """max over rows of max|a-b| / max|b| (b is the oracle)."""
    a = np.asarray(a, dtype=np.float64).reshape(-1, a.shape[-1])
    b = np.asarray(b, dtype=np.float64).reshape(-1, b.shape[-1])
    return float(np.max(np.abs(a - b).max(axis=1) / np.maximum(np.abs(b).max(axis=1), 1e-30)))


@dataclass
class LockstepReport:
    tokens: List[int] = field(default_factory=list)
    counts: List[int] = field(default_factory=list)
    near_ties: List[tuple] = field(default_factory=list)
    max_logit_err: float = 0.0
    max_hidden_err: float = 0.0
    max_kv_err: float = 0.0
    steps: int = 0
    decisions: int = 0

    @property
    def excused_fraction(self) -> float:
        return len(self.near_ties) / max(self.decisions, 1)


class StepTaps:
    """The debug taps of the CUDA path's last step, read once for the whole batch."""

    def __init__(self, gpu: SpecDecoder, g_tok, g_cnt, want_logits=True):
        self.T, self.g_tok, self.g_cnt = gpu.T, g_tok, g_cnt
        self.cand = gpu.debug(B.DBG_CAND)
        self.tok = gpu.debug(B.DBG_TOK).reshape(gpu.batch, gpu.T)
        self.pos = gpu.debug(B.DBG_POS).reshape(gpu.batch, gpu.T)
        self.logits = gpu.debug(B.DBG_LOGITS).reshape(gpu.batch, gpu.T, -1) if want_logits else None
        self.hidden = gpu.debug(B.DBG_HIDDEN).reshape(gpu.batch, gpu.T, -1)
        self.am = gpu.debug(B.DBG_ARGMAX).reshape(gpu.batch, gpu.T)
        self.path = gpu.debug(B.DBG_PATH)
        self.root = gpu.debug(B.DBG_NEXT_ROOT)
        self.seqlen = gpu.debug(B.DBG_SEQLEN)


class LockstepSeq:
    """One sequence's oracle and its comparison with the CUDA path, step by step."""

    def __init__(self, cfg, oracle: OracleSpecDecoder, seq: int, kmax: int, tol: float, tie_gap: float,
                 tie_from_row_error: bool = False, edge_tol: float = 1e-3, sample_tol: float = 1e-4):
        self.cfg, self.oracle, self.seq, self.kmax = cfg, oracle, seq, kmax
        self.tol, self.tie_gap, self.tie_from_row_error = tol, tie_gap, tie_from_row_error
        self.edge_tol, self.sample_tol = edge_tol, sample_tol
        self.rep = LockstepReport()

    # -- after both sides prefilled --
    def check_prefill(self, gpu: SpecDecoder):
        o, rep = self.oracle, self.rep
        h_gpu = gpu.debug(B.DBG_H_LAST)[self.seq]
        rep.max_hidden_err = max(rep.max_hidden_err, rel_err_rows(h_gpu[None], o.h_last[None]))
        assert rep.max_hidden_err <= self.tol, f"prefill hidden rel err {rep.max_hidden_err}"
        root_gpu = int(gpu.debug(B.DBG_NEXT_ROOT)[self.seq])
        if root_gpu != o.root_tok:
            lg = o.last_root_logits
            if o.sampling:
                self._excuse_sample(-1, lg, root_gpu)
            else:
                gap = float(lg[o.root_tok] - lg[root_gpu])
                assert gap < self.tie_gap, f"prefill root differs beyond a near-tie (gap {gap})"
                rep.near_ties.append((-1, 0, gap, o.root_tok, root_gpu))
            o.root_tok = root_gpu

    def _excuse_sample(self, step, logits_row, g_root):
        """The CUDA path drew another token at the same uniform: allowed only at a boundary of the
        cumulative distribution."""
        o = self.oracle
        z = np.asarray(logits_row, dtype=np.float64) / o.typ[2]
        w = np.exp(z - z.max())
        cdf = np.cumsum(w)
        target, total = o.last_u * cdf[-1], cdf[-1]
        lo = cdf[g_root - 1] if g_root > 0 else 0.0
        d = max(lo - target, target - cdf[g_root], 0.0) / total
        assert d <= self.sample_tol, f"step {step}: sampled root {g_root} is {d} of the total weight away from u"
        self.rep.near_ties.append((step, "sample", d, -1, g_root))

    # -- after the CUDA path ran one step; ov = the override table it was given (or None) --
    def after_gpu_step(self, taps: StepTaps, ov, gpu: Optional[SpecDecoder] = None, check_kv: bool = False):
        cfg, o, rep, b = self.cfg, self.oracle, self.rep, self.seq
        K, kmax, step = cfg.n_medusa, self.kmax, self.rep.steps
        g_cnt = int(taps.g_cnt[b])
        g_cand = taps.cand[b]
        # --- heads: candidate tables ---
        o_cand, z = o.candidates()
        if ov is not None:
            o_cand[1:, :kmax] = np.where(np.asarray(ov).reshape(K, kmax) < 0, o_cand[1:, :kmax], np.asarray(ov).reshape(K, kmax))
        use = None
        for k in range(K):
            kk = min(cfg.topk[k] if k < len(cfg.topk) else kmax, kmax)
            for j in range(kk):
                a, g = int(o_cand[k + 1, j]), int(g_cand[k + 1, j])
                rep.decisions += 1
                if a != g:
                    gap = abs(float(z[k][a] - z[k][g]))
                    bound = self.tie_gap
                    if self.tie_from_row_error:
                        # the CUDA path keeps no head logits to compare: a head's row is taken to be as far
                        # off as the worst logits / hidden row measured so far in this run
                        bound = max(bound, 2.0 * max(rep.max_logit_err, rep.max_hidden_err) * float(np.abs(z[k]).max()))
                    assert gap < bound, f"step {step}: head {k} rank {j} differs, gap {gap} (bound {bound})"
                    rep.near_ties.append((step, f"head{k}", gap, a, g))
                    use = g_cand
        if use is not None:
            ov_o = np.full((K, cfg.kmax), -1, dtype=np.int32)
            ov_o[:, :kmax] = g_cand[1:, :kmax]
            rec = o.step(ov_o)
        else:
            rec = o.step(None if ov is None else _pad_override(ov, K, kmax, cfg.kmax))
        # --- tree tokens, logits, hidden ---
        assert np.array_equal(taps.tok[b], rec["tok"]), f"step {step}: tree tokens differ"
        assert np.array_equal(taps.pos[b], rec["pos"]), f"step {step}: positions differ"
        lg_gpu, hd_gpu = taps.logits[b], taps.hidden[b]
        rep.max_logit_err = max(rep.max_logit_err, rel_err_rows(lg_gpu, rec["logits"]))
        rep.max_hidden_err = max(rep.max_hidden_err, rel_err_rows(hd_gpu, rec["hidden"]))
        assert rep.max_logit_err <= self.tol, f"step {step}: logits rel err {rep.max_logit_err}"
        assert rep.max_hidden_err <= self.tol, f"step {step}: hidden rel err {rep.max_hidden_err}"
        am_gpu = taps.am[b]
        tie_nodes = set()
        for v in range(len(am_gpu)):
            rep.decisions += 1
            if am_gpu[v] != rec["am"][v]:
                gap = float(rec["logits"][v][rec["am"][v]] - rec["logits"][v][am_gpu[v]])
                bound = self.tie_gap
                if self.tie_from_row_error:
                    bound = max(bound, 2.0 * float(np.abs(lg_gpu[v].astype(np.float64) - rec["logits"][v]).max()))
                assert gap < bound, f"step {step}: argmax at node {v} differs, gap {gap} (bound {bound})"
                tie_nodes.add(v)
                rep.near_ties.append((step, v, gap, int(rec["am"][v]), int(am_gpu[v])))
        # --- emitted tokens, accepted path, next root ---
        g_emit = [int(t) for t in taps.g_tok[b][:g_cnt]]
        o_emit = [int(t) for t in rec["tokens"]]
        g_root = int(taps.root[b])
        g_path = [int(v) for v in taps.path[b][:g_cnt]]
        o_path = [int(v) for v in rec["path"]]
        if g_path != o_path:
            # the deciding node: the last one both accepted paths share
            j = 0
            while j < min(len(g_path), len(o_path)) and g_path[j] == o_path[j]:
                j += 1
            assert j >= 1, f"step {step}: accepted paths do not share the root"
            u = o_path[j - 1]
            if o.accept_mode == "greedy":
                assert u in tie_nodes, (f"step {step}: accepted paths {g_path} vs oracle {o_path} part at node {u}, "
                                        f"which is no logged near tie")
            else:
                self._excuse_typical_edge(step, rec, u)
            o.force_commit(rec["n_before"], np.asarray(g_emit, dtype=np.int32), g_root)
            if g_root != rec["next_root"] and o.sampling:
                pass   # another last node: the draw came from another row; adopted above
        elif g_root != rec["next_root"]:
            assert g_emit == o_emit
            if o.sampling:
                self._excuse_sample(step, rec["logits"][rec["best"]], g_root)
            else:
                assert o_path[-1] in tie_nodes, f"step {step}: next root {g_root} vs oracle {rec['next_root']} without a near tie at node {o_path[-1]}"
            o.root_tok = g_root
        else:
            assert g_emit == o_emit
        assert int(taps.seqlen[b]) == o.n
        rep.tokens.extend(g_emit)
        rep.counts.append(g_cnt)
        rep.steps += 1
        if check_kv and gpu is not None:
            for l in sorted({0, cfg.n_layers - 1}):
                k, v = gpu.read_kv(b, l, 0, o.n)
                rep.max_kv_err = max(rep.max_kv_err, rel_err_rows(k.reshape(o.n, -1), o.cache.k[l, :o.n].reshape(o.n, -1)),
                                     rel_err_rows(v.reshape(o.n, -1), o.cache.v[l, :o.n].reshape(o.n, -1)))
            assert rep.max_kv_err <= self.tol, f"step {rep.steps}: cache rel err {rep.max_kv_err}"
        return rec

    def _excuse_typical_edge(self, step, rec, u):
        """Eq. 1 decided differently for a child of node u: allowed only if that child's probability
        is within edge_tol (relative) of the threshold."""
        o = self.oracle
        z = np.asarray(rec["logits"][u], dtype=np.float64) / o.typ[2]
        p = np.exp(z - z.max())
        p /= p.sum()
        thr = typical_threshold(p, o.typ[0], o.typ[1])
        kids = [v for v in range(len(o.parent)) if o.parent[v] == u]
        margins = [abs(float(p[rec["tok"][v]]) - thr) / thr for v in kids]
        assert margins and min(margins) <= self.edge_tol, f"step {step}: paths part at node {u}, Eq. 1 margins {margins}"
        self.rep.near_ties.append((step, f"edge@{u}", min(margins), -1, -1))


def run_lockstep(cfg, weights, tree, prompt, new_tokens: int, tol: float, tie_gap: float = 1e-2,
                 flags: int = 0, overrides: Optional[Callable] = None, max_seq: Optional[int] = None,
                 check_kv_every: int = 0, frag_token: int = -1, accept_mode: int = 0,
                 typ=(0.09, 0.3, 1.0), gpu: Optional[SpecDecoder] = None, oracle_model=None,
                 tie_from_row_error: bool = False, sampling: bool = False, seed: int = 0,
                 oracle: Optional[OracleSpecDecoder] = None, max_steps: Optional[int] = None) -> LockstepReport:
    """Single sequence. `oracle`: an already prefilled oracle decoder (its prefill is then not repeated)."""
    max_seq = max_seq or (len(prompt) + new_tokens + cfg.n_medusa + 2)
    prefilled = oracle is not None
    if oracle is None:
        model = oracle_model or OracleModel(cfg, weights)
        oracle = OracleSpecDecoder(model, tree, max_seq, frag_token=frag_token,
                                   accept_mode="typical" if accept_mode else "greedy",
                                   typ_eps=typ[0], typ_delta=typ[1], temperature=typ[2], sampling=sampling, seed=seed)
    own = gpu is None
    if own:
        gpu = SpecDecoder(cfg, upload_weights(cfg, weights), tree, max_seq, flags=flags | B.FLAG_KEEP_LOGITS,
                          frag_token=frag_token, accept_mode=accept_mode, typ_eps=typ[0], typ_delta=typ[1],
                          temperature=typ[2], sampling=sampling, seed=seed)
    ls = LockstepSeq(cfg, oracle, 0, gpu.kmax, tol, tie_gap, tie_from_row_error)
    try:
        if not prefilled:
            oracle.prefill(prompt)
        gpu.prefill(np.asarray(prompt, dtype=np.int32))
        ls.check_prefill(gpu)
        while len(ls.rep.tokens) < new_tokens and (max_steps is None or ls.rep.steps < max_steps):
            ov = overrides(ls.rep.steps, len(ls.rep.tokens)) if overrides else None
            g_tok, g_cnt = gpu.step(ov)
            kv = bool(check_kv_every) and (ls.rep.steps + 1) % check_kv_every == 0
            ls.after_gpu_step(StepTaps(gpu, g_tok, g_cnt), ov, gpu, check_kv=kv)
        st = gpu.debug(B.DBG_STATUS)
        assert st[0] == 0, f"device status {st}"
    finally:
        if own:
            gpu.close()
    return ls.rep


def run_lockstep_batch(cfg, gpu: SpecDecoder, oracles: Dict[int, OracleSpecDecoder], prompts, steps: int, tol: float,
                       tie_gap: float = 1e-2, tie_from_row_error: bool = False, check_kv: bool = True) -> Dict[int, LockstepReport]:
    """A batch on the CUDA path; `oracles` maps some sequence indices to (not yet prefilled) oracle
    decoders, each of which follows its own sequence in lock step."""
    seqs = {b: LockstepSeq(cfg, o, b, gpu.kmax, tol, tie_gap, tie_from_row_error) for b, o in oracles.items()}
    for b, o in oracles.items():
        o.prefill(prompts[b])
    gpu.prefill([np.asarray(p, dtype=np.int32) for p in prompts])
    for ls in seqs.values():
        ls.check_prefill(gpu)
    for _ in range(steps):
        g_tok, g_cnt = gpu.step()
        taps = StepTaps(gpu, g_tok, g_cnt)
        for ls in seqs.values():
            ls.after_gpu_step(taps, None, gpu, check_kv=check_kv)
    st = gpu.debug(B.DBG_STATUS)
    assert st[0] == 0, f"device status {st}"
    return {b: ls.rep for b, ls in seqs.items()}


def _pad_override(ov, K, kmax, kmax_cfg):
    out = np.full((K, kmax_cfg), -1, dtype=np.int32)
    out[:, :kmax] = np.asarray(ov, dtype=np.int32).reshape(K, kmax)
    return out
