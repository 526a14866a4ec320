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


def test_c2_controlled_draft_full_size(torch):
    """Configuration 2 at full size (32 layers, 512-token prompt, T = 64): with the controlled draft the
    emitted stream stays the plain greedy stream (lossless acceptance) up to a near tie of the base
    model's logits (a different draft changes tree slots and tile boundaries, hence float32 summation
    order), and the mean accepted length follows the closed form sum_i p^i within its sampling error."""
    from paper_2503_14153_b200 import SpecDecoder, build_tree
    from paper_2503_14153_b200 import binding as B
    from synthetic import controlled_draft, stream_weights_to_device
    cfg = get_config("c2")
    dw = stream_weights_to_device(cfg, "cuda:0", threads=16)
    tree = build_tree(cfg.topk, cfg.tree_nodes)
    prompt = draw_prompt(cfg)
    new_tokens = 256
    K = cfg.n_medusa
    dec = SpecDecoder(cfg, dw, tree, cfg.prompt_len + new_tokens + 16, flags=B.FLAG_KEEP_LOGITS)

    def generate(p, stream=None, want_gaps=False):
        dec.prefill(prompt)
        out, counts, gaps, step = [], [], [np.inf], 0
        uniforms, hit = (None, None) if p is None else controlled_draft(cfg, None, p, new_tokens)
        while len(out) < new_tokens:
            ov = None
            if p is not None:
                ov = uniforms[step].copy()
                for j in range(K):
                    pos = len(out) + 1 + j                # generated position head j predicts
                    if hit[step, j] and pos < len(stream):
                        ov[j, 0] = stream[pos]
                ov = ov[None, :, :dec.kmax]               # the library keeps only the ranks the tree uses
            tok, cnt = dec.step(ov)
            c = int(cnt[0])
            if want_gaps:
                # the token after path node v is the argmax of the logits row of v
                logits = dec.debug(B.DBG_LOGITS)
                for v in dec.debug(B.DBG_PATH)[0][:c]:
                    top2 = np.partition(logits[int(v)], -2)[-2:]
                    gaps.append(float(top2[1] - top2[0]))
            out.extend(int(t) for t in tok[0][:c])
            counts.append(c)
            step += 1
        return out, counts, gaps

    stream, _, gaps = generate(None, want_gaps=True)
    stream = stream + [0] * 8
    pooled = []                                                  # (count, expectation) of every step before a divergence
    for p in (0.3, 0.6, 0.9):
        out, counts, _ = generate(p, stream)
        n = min(new_tokens, len(out))
        k = next((i for i in range(n) if out[i] != stream[i]), n)
        if k < n:
            assert gaps[k] < TIE_GAP_32_LAYERS, f"p={p}: stream differs at {k} where the top-2 gap is {gaps[k]}"
        # steps that ended before the divergence follow the draft's statistics
        done, good = 0, []
        for c in counts[:-1]:
            done += c
            if done <= k:
                good.append(c)
        want = sum(p ** i for i in range(K + 1))
        pooled.extend((c, want) for c in good)
        if len(good) >= 8:
            got = float(np.mean(good))
            # counts lie in [1, K+1]: standard error at most (K/2)/sqrt(steps); allow 4 of them
            tol = 4 * (K / 2) / np.sqrt(len(good)) + 0.05
            assert abs(got - want) < tol, (p, got, want, tol)
            print(f"controlled draft p={p}: mean accepted length {got:.3f} (closed form {want:.3f}) over {len(good)} steps; "
                  f"stream identical for {k} of {n} tokens")
        else:
            print(f"controlled draft p={p}: near tie after {k} tokens ({len(good)} steps), counted in the pooled check only")
    # where a run met its near tie is a matter of rounding order: the pooled steps must still follow the closed forms
    assert len(pooled) >= 30, len(pooled)
    got, want = float(np.mean([c for c, _ in pooled])), float(np.mean([w for _, w in pooled]))
    assert abs(got - want) < 4 * (K / 2) / np.sqrt(len(pooled)) + 0.05, (got, want, len(pooled))
    dec.close()
