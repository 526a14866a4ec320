"""Pins of the oracle's decoder forward against things other than itself."""
import numpy as np
import pytest

from oracle.decoder import (KVCache, OracleModel, apply_rope, forward_full, forward_rows,
                            masked_attention, medusa_logits, rms_norm, rope_angles, top_k)
from oracle.numerics import round_bf16, silu
from synthetic import draw_weights, get_config

SMALL = get_config("c0", n_layers=2, d_model=64, n_heads=4, n_kv_heads=2, head_dim=16, d_ffn=96,
                   vocab=211, norm_gain="random", seed=7, rope_base=10000.0)


def test_rmsnorm_constant_vector_closed_form():
    # x = c everywhere -> mean(x^2) = c^2 -> y = c / sqrt(c^2 + eps) * g
    g = np.linspace(0.5, 1.5, 8)
    y = rms_norm(np.full((1, 8), 3.0), g, 1e-5)
    assert np.allclose(y[0], 3.0 / np.sqrt(9.0 + 1e-5) * g, rtol=0, atol=1e-15)


def test_rmsnorm_matches_torch():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(0)
    x, g = rng.standard_normal((5, 32)), rng.standard_normal(32)
    ref = torch.nn.functional.rms_norm(torch.from_numpy(x), (32,), torch.from_numpy(g), 1e-5).numpy()
    assert np.allclose(rms_norm(x, g, 1e-5), ref, atol=1e-13)


def test_rope_is_rotation_and_relative():
    rng = np.random.default_rng(1)
    D = 16
    q, k = rng.standard_normal((1, 1, D)), rng.standard_normal((1, 1, D))

    def rot(x, p):
        c, s = rope_angles(np.array([p]), D, 10000.0)
        return apply_rope(x, c, s)

    assert np.allclose(np.linalg.norm(rot(q, 37)), np.linalg.norm(q))
    a = (rot(q, 12) * rot(k, 5)).sum()
    b = (rot(q, 107) * rot(k, 100)).sum()
    assert np.isclose(a, b, atol=1e-12)
    assert np.allclose(rot(q, 0), q)
    # pair (0, D/2) rotates by angle pos * base^0 = pos
    e0 = np.zeros((1, 1, D)); e0[..., 0] = 1.0
    r = rot(e0, 2)
    assert np.isclose(r[0, 0, 0], np.cos(2.0)) and np.isclose(r[0, 0, D // 2], np.sin(2.0))
    # pair (1, D/2+1) rotates by pos * base^(-2/D)
    e1 = np.zeros((1, 1, D)); e1[..., 1] = 1.0
    r = rot(e1, 3)
    th = 3.0 * 10000.0 ** (-2.0 / D)
    assert np.isclose(r[0, 0, 1], np.cos(th)) and np.isclose(r[0, 0, D // 2 + 1], np.sin(th))


def test_attention_equal_keys_is_mean_of_visible_values():
    rng = np.random.default_rng(2)
    T, S, H, D = 3, 6, 2, 8
    q = rng.standard_normal((T, H, D))
    k = np.tile(rng.standard_normal((1, H, D)), (S, 1, 1))
    v = rng.standard_normal((S, H, D))
    vis = np.zeros((T, S), dtype=bool)
    vis[0, :2] = True; vis[1, [0, 3, 5]] = True; vis[2, :] = True
    o = masked_attention(q, k, v, vis, lambda x: x)
    for t in range(T):
        assert np.allclose(o[t], v[vis[t]].mean(axis=0), atol=1e-13)


def test_attention_matches_torch_sdpa_with_gqa():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(3)
    T, S, H, Hkv, D = 5, 9, 4, 2, 8
    q, k, v = rng.standard_normal((T, H, D)), rng.standard_normal((S, Hkv, D)), rng.standard_normal((S, Hkv, D))
    vis = rng.random((T, S)) < 0.6
    vis[:, 0] = True
    o = masked_attention(q, k, v, vis, lambda x: x)
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]
    tk = torch.from_numpy(np.repeat(k, H // Hkv, axis=1)).permute(1, 0, 2)[None]
    tv = torch.from_numpy(np.repeat(v, H // Hkv, axis=1)).permute(1, 0, 2)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=torch.from_numpy(vis))
    assert np.allclose(o, ref[0].permute(1, 0, 2).numpy(), atol=1e-12)


def test_silu_closed_values():
    assert silu(np.array([0.0]))[0] == 0.0
    assert np.isclose(silu(np.array([1.0]))[0], 1.0 / (1.0 + np.exp(-1.0)))
    assert np.isclose(silu(np.array([-30.0]))[0], -30.0 * np.exp(-30.0), rtol=1e-9)


def test_round_bf16_matches_torch_and_ties_to_even():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(4)
    x = np.concatenate([rng.standard_normal(4096) * 10.0 ** rng.integers(-6, 6, 4096),
                        np.array([1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, 0.0, -0.0, 1e-40, 3.3895e38])]).astype(np.float32)
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(round_bf16(x).astype(np.float32), ref)
    assert round_bf16(np.array([1.0 + 2 ** -8]))[0] == 1.0          # tie -> even mantissa
    assert round_bf16(np.array([1.0 + 3 * 2 ** -8]))[0] == 1.0 + 2 ** -6


def test_topk_matches_full_sort_and_breaks_ties_low():
    rng = np.random.default_rng(5)
    v = rng.standard_normal(1000).astype(np.float32)
    v[[10, 700]] = v.max() + 1.0                       # exact tie at the top
    ref = sorted(range(1000), key=lambda i: (-float(v[i]), i))[:7]
    assert list(top_k(v, 7)) == ref
    assert list(top_k(v, 2)) == [10, 700]


def test_medusa_head_zero_matrix_closed_form():
    cfg = SMALL.with_(n_medusa=1, topk=(3,))
    w = draw_weights(cfg)
    w["medusa.0.w"] = np.zeros_like(w["medusa.0.w"])
    m = OracleModel(cfg, w)
    h = np.random.default_rng(6).standard_normal(cfg.d_model)
    z = medusa_logits(m, h)
    r = h + silu(w["medusa.0.b"].astype(np.float64))
    assert np.allclose(z[0], (w["lm_head"].astype(np.float64) @ r).astype(np.float32), rtol=1e-6, atol=1e-7)


def _hf_model(cfg, w):
    torch = pytest.importorskip("torch")
    transformers = pytest.importorskip("transformers")
    hf_cfg = transformers.LlamaConfig(
        vocab_size=cfg.vocab, hidden_size=cfg.d_model, intermediate_size=cfg.d_ffn,
        num_hidden_layers=cfg.n_layers, num_attention_heads=cfg.n_heads,
        num_key_value_heads=cfg.n_kv_heads, head_dim=cfg.head_dim, rms_norm_eps=cfg.rms_eps,
        rope_theta=cfg.rope_base, max_position_embeddings=512, tie_word_embeddings=False,
        attention_bias=False, mlp_bias=False, hidden_act="silu")
    hf_cfg._attn_implementation = "eager"
    model = transformers.LlamaForCausalLM(hf_cfg).to(torch.float64).eval()
    sd = {"model.embed_tokens.weight": w["embed"], "lm_head.weight": w["lm_head"],
          "model.norm.weight": w["final_norm"]}
    names = {"attn_norm": "input_layernorm.weight", "wq": "self_attn.q_proj.weight",
             "wk": "self_attn.k_proj.weight", "wv": "self_attn.v_proj.weight",
             "wo": "self_attn.o_proj.weight", "ffn_norm": "post_attention_layernorm.weight",
             "w_gate": "mlp.gate_proj.weight", "w_up": "mlp.up_proj.weight", "w_down": "mlp.down_proj.weight"}
    for l in range(cfg.n_layers):
        for k, v in names.items():
            sd[f"model.layers.{l}.{v}"] = w[f"layers.{l}.{k}"]
    missing, unexpected = model.load_state_dict({k: torch.from_numpy(v).to(torch.float64) for k, v in sd.items()},
                                                strict=False)
    assert not unexpected and all("rotary" in m or "inv_freq" in m for m in missing), (missing, unexpected)
    return model, torch


def test_forward_matches_transformers_llama():
    """Whole forward (RoPE pairing, GQA mapping, norm placement, SwiGLU, untied lm_head)
    against the transformers library's Llama on a small shape with random gains."""
    cfg = SMALL
    w = draw_weights(cfg)
    model, torch = _hf_model(cfg, w)
    toks = np.random.default_rng(8).integers(0, cfg.vocab, 23)
    with torch.no_grad():
        ref = model(torch.from_numpy(toks)[None]).logits[0].numpy()
    got = forward_full(OracleModel(cfg, w), toks)
    assert np.abs(got - ref).max() <= 2e-6 * np.abs(ref).max()   # float32 rounding of the logits


def test_cached_forward_equals_recompute(tiny_cfg, tiny_weights):
    m = OracleModel(tiny_cfg, tiny_weights)
    toks = np.random.default_rng(9).integers(0, tiny_cfg.vocab, 20)
    full = forward_full(m, toks)
    cache = KVCache(tiny_cfg, 32)
    n = 0
    for chunk in (toks[:7], toks[7:8], toks[8:20]):
        c = len(chunk)
        _, lg = forward_rows(m, cache, n, chunk, np.arange(n, n + c), np.tril(np.ones((c, c), bool)))
        assert np.abs(lg - full[n:n + c]).max() < 1e-6
        n += c


def test_tree_rows_equal_per_path_recompute(tiny_cfg, tiny_weights):
    """A tree node's logits equal the no-cache logits of prompt + the node's root path."""
    from oracle.tree import ancestor_mask, build_tree
    m = OracleModel(tiny_cfg, tiny_weights)
    rng = np.random.default_rng(10)
    prompt = rng.integers(0, tiny_cfg.vocab, 9)
    tree = build_tree((3, 2, 2), 10)
    tok = rng.integers(0, tiny_cfg.vocab, 10)
    cache = KVCache(tiny_cfg, 32)
    forward_rows(m, cache, 0, prompt, np.arange(9), np.tril(np.ones((9, 9), bool)))
    _, lg = forward_rows(m, cache, 9, tok, 9 + tree["depth"], ancestor_mask(tree["parent"]))
    for v in (0, 3, 7, 9):
        path, u = [], v
        while u >= 0:
            path.append(u); u = int(tree["parent"][u])
        seq = np.concatenate([prompt, tok[path[::-1]]])
        assert np.abs(forward_full(m, seq)[-1] - lg[v]).max() < 1e-6


def test_bf16_mode_stays_close_to_exact():
    cfg = SMALL.with_(dtype="bf16")
    w = draw_weights(cfg)
    toks = np.random.default_rng(11).integers(0, cfg.vocab, 12)
    a = forward_full(OracleModel(cfg, w), toks)
    wq = {k: (round_bf16(v).astype(np.float32) if v.ndim == 2 or ".b" in k else v) for k, v in w.items()}
    b = forward_full(OracleModel(cfg.with_(dtype="fp32"), wq), toks)
    assert np.abs(a - b).max() <= 2e-2 * np.abs(b).max()
    assert np.abs(a - b).max() > 0


def _head_only_model(d, V, W, b, lm):
    """An OracleModel that holds just one extra head and the lm_head (all medusa_logits reads)."""
    cfg = SMALL.with_(d_model=d, vocab=V, n_medusa=1, topk=(1,), dtype="fp32")
    return OracleModel(cfg, {"medusa.0.w": np.asarray(W, np.float32), "medusa.0.b": np.asarray(b, np.float32),
                             "lm_head": np.asarray(lm, np.float32)})


def test_medusa_head_hand_worked_2x2():
    """Extra head on the last hidden state (Sec. III-B, model architecture): residual block
    h + SiLU(W h + b) with W stored [out, in], then the shared lm_head. Worked by hand:
    W = [[1, 2], [0, -1]], b = (0, 1), h = (1, 1): W h + b = (3, 0), SiLU -> (3 / (1 + e^-3), 0),
    r = (1 + 3 / (1 + e^-3), 1); lm_head = [[0, 1], [1, 0], [1, 1]] -> z = (r1, r0, r0 + r1).
    With W transposed W^T h + b = (1, 2) and z differs in every entry."""
    m = _head_only_model(2, 3, [[1, 2], [0, -1]], [0, 1], [[0, 1], [1, 0], [1, 1]])
    z = medusa_logits(m, np.array([1.0, 1.0]))
    r0 = 1.0 + 3.0 / (1.0 + np.exp(-3.0))
    assert np.allclose(z[0], [1.0, r0, r0 + 1.0], rtol=1e-6)


def test_medusa_head_matches_torch_linear_modules():
    """The same block written with torch.nn.Linear modules in float64 (weight [out, in], x W^T + b)
    on a random, non-symmetric head matrix: a transposed matrix, a dropped bias or residual,
    or the lm_head applied to the wrong vector fails."""
    torch = pytest.importorskip("torch")
    cfg = SMALL.with_(n_medusa=3, topk=(3, 2, 2))
    w = draw_weights(cfg)
    for k in range(3):                                   # N(0, 0.02) would make SiLU nearly linear: scale up
        w[f"medusa.{k}.w"] = (w[f"medusa.{k}.w"] * 40.0).astype(np.float32)
        w[f"medusa.{k}.b"] = (w[f"medusa.{k}.b"] * 20.0).astype(np.float32)
    h = np.random.default_rng(12).standard_normal(cfg.d_model)
    z = medusa_logits(OracleModel(cfg, w), h)
    lm = torch.nn.Linear(cfg.d_model, cfg.vocab, bias=False, dtype=torch.float64)
    th = torch.from_numpy(h)
    with torch.no_grad():
        lm.weight.copy_(torch.from_numpy(w["lm_head"]).double())
        for k in range(3):
            blk = torch.nn.Linear(cfg.d_model, cfg.d_model, bias=True, dtype=torch.float64)
            blk.weight.copy_(torch.from_numpy(w[f"medusa.{k}.w"]).double())
            blk.bias.copy_(torch.from_numpy(w[f"medusa.{k}.b"]).double())
            ref = lm(th + torch.nn.functional.silu(blk(th))).numpy()
            assert np.abs(z[k] - ref).max() <= 2e-6 * np.abs(ref).max()      # float32 rounding of z
            wrong = lm(th + torch.nn.functional.silu(th @ blk.weight + blk.bias)).numpy()
            assert np.abs(z[k] - wrong).max() > 1e-2 * np.abs(ref).max()     # the transposed reading is far away


def test_prefill_across_chunk_boundaries_equals_full_forward():
    """OracleSpecDecoder.prefill walks the prompt in chunks; a 150-token prompt in chunks of 32
    (four full chunks and a ragged one) must leave the first root token, its logits and the
    cache rows of the plain causal forward over the whole prompt."""
    from oracle.spec import OracleSpecDecoder
    from oracle.tree import build_tree
    cfg = SMALL
    m = OracleModel(cfg, draw_weights(cfg))
    prompt = np.random.default_rng(13).integers(0, cfg.vocab, 150)
    full = forward_full(m, prompt)
    dec = OracleSpecDecoder(m, build_tree((2, 2, 2), 6), 200)
    dec.prefill(prompt, chunk=32)
    assert dec.n == 150
    assert np.abs(dec.last_root_logits - full[-1]).max() <= 1e-6 * np.abs(full[-1]).max()
    assert dec.root_tok == int(np.argmax(full[-1].astype(np.float32)))
    # a later row sees every earlier chunk: the next token's logits after one more cached row
    one = KVCache(cfg, 151)
    forward_rows(m, one, 0, prompt, np.arange(150), np.tril(np.ones((150, 150), bool)))
    for l in range(cfg.n_layers):
        assert np.allclose(dec.cache.k[l, :150], one.k[l, :150], atol=1e-12)
        assert np.allclose(dec.cache.v[l, :150], one.v[l, :150], atol=1e-12)
    ext = np.concatenate([prompt, [dec.root_tok]])
    _, lg = forward_rows(m, dec.cache, 150, [dec.root_tok], [150], np.ones((1, 1), bool))
    ref = forward_full(m, ext)[-1]
    assert np.abs(lg[0] - ref).max() <= 1e-6 * np.abs(ref).max()
