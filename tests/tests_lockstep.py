"""Lock-step comparison of the CUDA decode loop with the CPU oracle (test harness).

Both decoders advance one step at a time from the same committed prefix. Token decisions
must agree exactly except at logged near-ties (the oracle's gap between the two competing
logits is below `tie_gap`), where the oracle adopts the CUDA path's decision and the run
continues. Logits and hidden states are compared per row with
max|a-b| / max|b| <= tol.
"""
from dataclasses import dataclass, field
from typing import Callable, List, Optional

import numpy as np

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


def run_lockstep(cfg, weights, tree, prompt, new_tokens: int, tol: float, tie_gap: float = 1e-2,
                 flags: int = 0, overrides: Optional[Callable] = None, max_seq: Optional[int] = None,
                 check_kv_every: int = 0, frag_token: int = -1, accept_mode: int = 0,
                 typ=(0.09, 0.3, 1.0), gpu: Optional[SpecDecoder] = None, oracle_model=None) -> LockstepReport:
    max_seq = max_seq or (len(prompt) + new_tokens + cfg.n_medusa + 2)
    model = oracle_model or OracleModel(cfg, weights)
    oracle = OracleSpecDecoder(model, tree, max_seq, frag_token=frag_token,
                               accept_mode="typical" if accept_mode else "greedy",
                               typ_eps=typ[0], typ_delta=typ[1], temperature=typ[2])
    own = gpu is None
    if own:
        gpu = SpecDecoder(cfg, upload_weights(cfg, weights), tree, max_seq, flags=flags | B.FLAG_KEEP_LOGITS,
                          frag_token=frag_token, accept_mode=accept_mode, typ_eps=typ[0], typ_delta=typ[1],
                          temperature=typ[2])
    rep = LockstepReport()
    K, kmax = cfg.n_medusa, gpu.kmax
    try:
        oracle.prefill(prompt)
        gpu.prefill(np.asarray(prompt, dtype=np.int32))
        h_gpu = gpu.debug(B.DBG_H_LAST)[0]
        rep.max_hidden_err = max(rep.max_hidden_err, rel_err_rows(h_gpu[None], oracle.h_last[None]))
        assert rep.max_hidden_err <= tol, f"prefill hidden rel err {rep.max_hidden_err}"
        root_gpu = int(gpu.debug(B.DBG_NEXT_ROOT)[0])
        if root_gpu != oracle.root_tok:
            lg = oracle.last_root_logits
            gap = float(lg[oracle.root_tok] - lg[root_gpu])
            assert gap < tie_gap, f"prefill root differs beyond a near-tie (gap {gap})"
            rep.near_ties.append((-1, 0, gap, oracle.root_tok, root_gpu))
            oracle.root_tok = root_gpu
        while len(rep.tokens) < new_tokens:
            ov = overrides(rep.steps, len(rep.tokens)) if overrides else None
            g_tok, g_cnt = gpu.step(ov)
            g_tok, g_cnt = g_tok[0], int(g_cnt[0])
            g_cand = gpu.debug(B.DBG_CAND)[0]
            # --- heads: candidate tables ---
            o_cand, z = oracle.candidates()
            if ov is not None:
                o_cand[1:, :kmax] = np.where(np.asarray(ov).reshape(K, kmax) < 0, o_cand[1:, :kmax],
                                             np.asarray(ov).reshape(K, kmax))
            use = None
            for k in range(K):
                kk = cfg.topk[k] if k < len(cfg.topk) else kmax
                kk = min(kk, kmax)
                for j in range(kk):
                    a, b = int(o_cand[k + 1, j]), int(g_cand[k + 1, j])
                    rep.decisions += 1
                    if a != b:
                        gap = abs(float(z[k][a] - z[k][b]))
                        assert gap < tie_gap, f"step {rep.steps}: head {k} rank {j} differs, gap {gap}"
                        rep.near_ties.append((rep.steps, f"head{k}", gap, a, b))
                        use = g_cand
            if use is not None:
                ov_o = np.full((K, cfg.kmax), -1, dtype=np.int32)
                ov_o[:, :kmax] = g_cand[1:, :kmax]
                rec = oracle.step(ov_o)
            else:
                rec = oracle.step(None if ov is None else _pad_override(ov, K, kmax, cfg.kmax))
            # --- tree tokens, logits, hidden ---
            assert np.array_equal(gpu.debug(B.DBG_TOK), rec["tok"]), f"step {rep.steps}: tree tokens differ"
            assert np.array_equal(gpu.debug(B.DBG_POS), rec["pos"]), f"step {rep.steps}: positions differ"
            lg_gpu = gpu.debug(B.DBG_LOGITS)
            hd_gpu = gpu.debug(B.DBG_HIDDEN)
            rep.max_logit_err = max(rep.max_logit_err, rel_err_rows(lg_gpu, rec["logits"]))
            rep.max_hidden_err = max(rep.max_hidden_err, rel_err_rows(hd_gpu, rec["hidden"]))
            assert rep.max_logit_err <= tol, f"step {rep.steps}: logits rel err {rep.max_logit_err}"
            assert rep.max_hidden_err <= tol, f"step {rep.steps}: hidden rel err {rep.max_hidden_err}"
            am_gpu = gpu.debug(B.DBG_ARGMAX)
            tie_nodes = set()
            for v in range(len(am_gpu)):
                rep.decisions += 1
                if am_gpu[v] != rec["am"][v]:
                    gap = float(rec["logits"][v][rec["am"][v]] - rec["logits"][v][am_gpu[v]])
                    assert gap < tie_gap, f"step {rep.steps}: argmax at node {v} differs, gap {gap}"
                    tie_nodes.add(v)
                    rep.near_ties.append((rep.steps, v, gap, int(rec["am"][v]), int(am_gpu[v])))
            # --- emitted tokens ---
            g_emit = [int(t) for t in g_tok[:g_cnt]]
            o_emit = [int(t) for t in rec["tokens"]]
            g_root = int(gpu.debug(B.DBG_NEXT_ROOT)[0])
            if g_emit != o_emit or g_root != rec["next_root"]:
                assert tie_nodes, f"step {rep.steps}: emitted {g_emit}+{g_root} vs oracle {o_emit}+{rec['next_root']}"
                oracle.force_commit(rec["n_before"], np.asarray(g_emit, dtype=np.int32), g_root)
            else:
                assert np.array_equal(gpu.debug(B.DBG_PATH)[0][:g_cnt], rec["path"])
            assert int(gpu.debug(B.DBG_SEQLEN)[0]) == oracle.n
            rep.tokens.extend(g_emit)
            rep.counts.append(g_cnt)
            rep.steps += 1
            if check_kv_every and rep.steps % check_kv_every == 0:
                for l in sorted({0, cfg.n_layers - 1}):
                    k, v = gpu.read_kv(0, l, 0, oracle.n)
                    rep.max_kv_err = max(rep.max_kv_err, rel_err_rows(k.reshape(oracle.n, -1), oracle.cache.k[l, :oracle.n].reshape(oracle.n, -1)),
                                         rel_err_rows(v.reshape(oracle.n, -1), oracle.cache.v[l, :oracle.n].reshape(oracle.n, -1)))
                assert rep.max_kv_err <= tol, f"step {rep.steps}: cache rel err {rep.max_kv_err}"
        st = gpu.debug(B.DBG_STATUS)
        assert st[0] == 0, f"device status {st}"
    finally:
        if own:
            gpu.close()
    return rep


def _pad_override(ov, K, kmax, kmax_cfg):
    out = np.full((K, kmax_cfg), -1, dtype=np.int32)
    out[:, :kmax] = np.asarray(ov, dtype=np.int32).reshape(K, kmax)
    return out
