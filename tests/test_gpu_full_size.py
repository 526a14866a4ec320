"""Parity at the benchmark's own sizes (needs a B200 and tens of GB of host memory).

The element-by-element tests in test_gpu_parity.py use shapes the CPU oracle finishes in seconds.
Here the CUDA path runs in the launch configuration bench.py times (7B shape, T = 64, 296 persistent
GEMM CTAs, two CTAs per SM) and is compared with the oracle where the oracle can still follow:
one full 32-layer draft-and-verify step after a short prompt; the long-context and batched
configurations on the 7B shape cut to two layers.
"""
import numpy as np
import pytest

from synthetic import draw_prompt, draw_prompt_batch, draw_weights, get_config

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2
# At 32 layers the max-norm error of a hidden row is dominated by single bf16 roundings that flip
# and are then amplified layer by layer: two equally valid float32 summation orders of the CUDA
# path itself (296 against 148 GEMM CTAs) already differ by 0.7% / 1.1% / 1.6% / 2.3% of a row's
# largest value at 4 / 8 / 16 / 32 layers of this random-weight model. The 2e-2 bound therefore
# holds up to about 16 layers; the full-depth comparison uses twice that.
TOL_BF16_32_LAYERS = 4e-2
TIE_GAP = 1e-2
# A logits row that is off by up to 4e-2 of its largest magnitude (about 5 with these weights) can
# swap two candidates whose logits are closer than that error: at full depth a token decision may
# differ from the oracle's where the oracle's gap is below 0.2; every such case is logged.
TIE_GAP_32_LAYERS = 0.2


@pytest.fixture(scope="module")
def torch():
    t = pytest.importorskip("torch")
    if not t.cuda.is_available():
        pytest.skip("no CUDA device")
    return t


def test_c1_7b_shape_full_depth_one_step_vs_oracle(torch):
    """Configuration 1 at full depth: heads, tree, 32-layer verify forward, acceptance, compaction of one
    step, every decision and every logits / hidden row against the oracle."""
    from paper_2503_14153_b200 import build_tree
    from tests_lockstep import run_lockstep
    cfg = get_config("c1")
    w = draw_weights(cfg, threads=16)
    tree = build_tree(cfg.topk, cfg.tree_nodes)
    rep = run_lockstep(cfg, w, tree, draw_prompt(cfg, 16), 1, TOL_BF16_32_LAYERS, TIE_GAP_32_LAYERS, check_kv_every=1)
    assert rep.steps == 1 and rep.max_logit_err < TOL_BF16_32_LAYERS and rep.max_hidden_err < TOL_BF16_32_LAYERS
    print(f"full depth: logits rel err {rep.max_logit_err:.4f}, hidden {rep.max_hidden_err:.4f}, cache {rep.max_kv_err:.4f}, near-ties {len(rep.near_ties)}")


def test_c3_long_context_two_layers_vs_oracle(torch):
    """Configuration 3 (8192 cached positions, T = 128) on the 7B shape cut to two layers: KV splits,
    tiles fetched ahead of the dependency, the merge of the splits and the tree mask at the cache's end."""
    from paper_2503_14153_b200 import build_tree
    from tests_lockstep import run_lockstep
    cfg = get_config("c3", n_layers=2, tree_nodes=128)
    w = draw_weights(cfg, threads=16)
    tree = build_tree(cfg.topk, cfg.tree_nodes)
    # 8192 keys per row: the kernel rounds each probability to bf16 relative to the running maximum of
    # its tile sequence, the oracle relative to the row's global maximum; both are roundings of the same
    # numbers at 2^-9, but not the same roundings, so candidates closer than 5e-2 may swap
    rep = run_lockstep(cfg, w, tree, draw_prompt(cfg), 2, TOL_BF16, 5e-2)
    print(f"long context: logits rel err {rep.max_logit_err:.4f}, hidden {rep.max_hidden_err:.4f}, near-ties {len(rep.near_ties)}")
    assert rep.steps >= 1 and rep.max_logit_err < TOL_BF16


def test_c3_stream_does_not_depend_on_tree_size(torch):
    """Greedy acceptance is lossless: at 2048 cached positions the emitted stream is the same for
    T = 16, 32, 64 and 128 (two layers of the 7B shape; CUDA path only)."""
    from paper_2503_14153_b200 import SpecDecoder, build_tree, upload_weights
    from paper_2503_14153_b200 import binding as B
    cfg = get_config("c3", n_layers=2, prompt_len=2048)
    w = draw_weights(cfg, threads=16)
    dw = upload_weights(cfg, w)
    prompt = draw_prompt(cfg)
    streams, hidden = [], []
    for T in (16, 32, 64, 128):
        dec = SpecDecoder(cfg, dw, build_tree(cfg.topk, T), cfg.prompt_len + 64)
        dec.prefill(prompt)
        out = []
        while len(out) < 12:
            tok, cnt = dec.step()
            out.extend(int(t) for t in tok[0][: int(cnt[0])])
        streams.append(out[:12])
        hidden.append(dec.debug(B.DBG_H_LAST)[0].copy())
        dec.close()
    # identical unless a near-tie flipped (different T = different GEMM tiling = different rounding)
    base = streams[-1]
    for s in streams[:-1]:
        k = next((i for i, (a, b) in enumerate(zip(s, base)) if a != b), len(base))
        assert k >= 8, (streams, "streams diverge early: not a near-tie")


def test_c4_batch16_matches_single_sequence_runs(torch):
    """Configuration 4 (16 ragged prompts, M = 16 x 64 = 1024 rows) on two layers of the 7B shape: every
    sequence of the batch emits what it emits when decoded alone, and its last hidden state agrees."""
    from paper_2503_14153_b200 import SpecDecoder, build_tree, upload_weights
    from paper_2503_14153_b200 import binding as B
    cfg = get_config("c4", n_layers=2)
    w = draw_weights(cfg, threads=16)
    dw = upload_weights(cfg, w)
    prompts = draw_prompt_batch(cfg, 16, 128, 2048)
    tree = build_tree(cfg.topk, cfg.tree_nodes)
    steps = 4
    dec = SpecDecoder(cfg, dw, tree, 2048 + 64, max_batch=16)
    dec.prefill(prompts)
    emitted = [[] for _ in prompts]
    for _ in range(steps):
        tok, cnt = dec.step()
        for b in range(16):
            emitted[b].extend(int(t) for t in tok[b][: int(cnt[b])])
    h_batch = dec.debug(B.DBG_H_LAST).copy()
    assert dec.debug(B.DBG_STATUS)[0] == 0
    dec.close()
    for b in (0, 7, 15):
        one = SpecDecoder(cfg, dw, tree, 2048 + 64, max_batch=1)
        one.prefill(prompts[b])
        out = []
        for _ in range(steps):
            tok, cnt = one.step()
            out.extend(int(t) for t in tok[0][: int(cnt[0])])
        h_one = one.debug(B.DBG_H_LAST)[0].copy()
        one.close()
        k = next((i for i, (x, y) in enumerate(zip(out, emitted[b])) if x != y), min(len(out), len(emitted[b])))
        if k == min(len(out), len(emitted[b])) and len(out) == len(emitted[b]):
            err = np.abs(h_one - h_batch[b]).max() / np.abs(h_one).max()
            assert err < TOL_BF16, (b, err)
        else:
            assert k >= 2, (b, out, emitted[b])
