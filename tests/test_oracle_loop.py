"""Whole-loop pins: the draft-and-verify stream equals plain no-cache greedy decoding."""
import numpy as np
import pytest

from oracle.decoder import KVCache, OracleModel, forward_rows
from oracle.spec import OracleSpecDecoder, greedy_decode_nocache
from oracle.tree import build_tree, chain_tree
from synthetic import controlled_draft, draw_prompt, draw_weights, get_config


@pytest.fixture(scope="module")
def tiny(tiny_cfg, tiny_weights):
    model = OracleModel(tiny_cfg, tiny_weights)
    prompt = draw_prompt(tiny_cfg)
    ref = greedy_decode_nocache(model, prompt, 40)
    return model, prompt, ref


def test_chain_tree_equals_autoregressive_greedy(tiny):
    model, prompt, ref = tiny
    dec = OracleSpecDecoder(model, chain_tree(model.cfg.n_medusa + 1), 128)
    out, counts = dec.generate(prompt, 40)
    assert np.array_equal(out, ref)
    assert all(1 <= c <= model.cfg.n_medusa + 1 for c in counts)


@pytest.mark.parametrize("T", [1, 5, 16])
def test_stream_independent_of_tree_size(tiny, T):
    model, prompt, ref = tiny
    dec = OracleSpecDecoder(model, build_tree(model.cfg.topk, T), 128)
    out, _ = dec.generate(prompt, 40)
    assert np.array_equal(out, ref)


def test_single_node_tree_emits_one_token_per_step(tiny):
    model, prompt, ref = tiny
    dec = OracleSpecDecoder(model, build_tree(model.cfg.topk, 1), 128)
    out, counts = dec.generate(prompt, 10)
    assert counts == [1] * 10 and np.array_equal(out, ref[:10])


def test_stream_independent_of_draft_and_accept_length_closed_form(tiny):
    """Controlled draft: head j's rank-0 candidate is the true greedy token with
    probability p, so E[count] = sum_i p^i (i = 0..K) up to chance matches."""
    model, prompt, ref = tiny
    cfg = model.cfg
    long_ref = OracleSpecDecoder(model, chain_tree(1), 256).generate(prompt, 140)[0]
    assert np.array_equal(long_ref[:40], ref)
    for p in (0.0, 0.6, 1.0):
        uniforms, hit = controlled_draft(cfg, long_ref, p, 200)

        def ov(i, done, dec):
            t = uniforms[i].copy()
            for j in range(cfg.n_medusa):
                if hit[i, j]:
                    t[j, 0] = long_ref[done + 1 + j]
            return t

        dec = OracleSpecDecoder(model, build_tree(cfg.topk, cfg.tree_nodes), 256)
        out, counts = dec.generate(prompt, 130, overrides=ov)
        assert np.array_equal(out, long_ref[:130])
        expect = sum(p ** i for i in range(cfg.n_medusa + 1))
        mean = np.mean(counts[:-1])
        if p in (0.0, 1.0):
            assert mean == pytest.approx(expect, abs=0.05)
        else:
            assert abs(mean - expect) < 4 * 1.2 / np.sqrt(len(counts))


def test_cache_after_compaction_equals_fresh_prefill(tiny):
    model, prompt, _ = tiny
    cfg = model.cfg
    dec = OracleSpecDecoder(model, build_tree(cfg.topk, cfg.tree_nodes), 128)
    dec.prefill(prompt)
    emitted = []
    for _ in range(24):
        emitted.extend(int(t) for t in dec.step()["tokens"])
    fresh = KVCache(cfg, 128 + cfg.tree_nodes)
    seq = np.concatenate([prompt, np.asarray(emitted, dtype=np.int32)])
    forward_rows(model, fresh, 0, seq, np.arange(len(seq)), np.tril(np.ones((len(seq),) * 2, bool)), [0])
    assert dec.n == len(seq)
    assert np.abs(dec.cache.k[:, :dec.n] - fresh.k[:, :dec.n]).max() < 1e-9
    assert np.abs(dec.cache.v[:, :dec.n] - fresh.v[:, :dec.n]).max() < 1e-9


def test_force_commit_reproduces_own_step(tiny):
    model, prompt, _ = tiny
    cfg = model.cfg
    a = OracleSpecDecoder(model, build_tree(cfg.topk, cfg.tree_nodes), 128)
    b = OracleSpecDecoder(model, build_tree(cfg.topk, cfg.tree_nodes), 128)
    a.prefill(prompt); b.prefill(prompt)
    for _ in range(6):
        rec = a.step()
        b.force_commit(rec["n_before"], rec["tokens"], rec["next_root"])
        assert b.n == a.n and b.root_tok == a.root_tok
        assert np.abs(b.h_last - a.h_last).max() < 1e-9
        assert np.abs(b.cache.k[:, :b.n] - a.cache.k[:, :a.n]).max() < 1e-9


def test_fragment_truncation_keeps_stream_and_ends_spans_on_marker(tiny):
    model, prompt, ref = tiny
    cfg = model.cfg
    frag = int(np.bincount(ref).argmax())
    dec = OracleSpecDecoder(model, build_tree(cfg.topk, cfg.tree_nodes), 128, frag_token=frag)
    dec.prefill(prompt)
    out = []
    for _ in range(30):
        rec = dec.step()
        toks = [int(t) for t in rec["tokens"]]
        assert len(toks) == 1 or toks[-1] == frag
        out.extend(toks)
    assert np.array_equal(np.asarray(out[:40]), ref[:len(out[:40])])


def test_bf16_small_model_is_lossless_too():
    cfg = get_config("c0", n_layers=2, d_model=64, n_heads=4, n_kv_heads=2, head_dim=16, d_ffn=96,
                     vocab=300, dtype="bf16", seed=12, norm_gain="random")
    model = OracleModel(cfg, draw_weights(cfg))
    prompt = draw_prompt(cfg, 10)
    ref = greedy_decode_nocache(model, prompt, 24)
    out, _ = OracleSpecDecoder(model, build_tree(cfg.topk, 16), 64).generate(prompt, 24)
    assert np.array_equal(out, ref)
