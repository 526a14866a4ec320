"""Parity of the CUDA decode loop with the CPU oracle, through the C ABI (needs a B200)."""
import numpy as np
import pytest

from synthetic import controlled_draft, draw_prompt, draw_weights, get_config

pytestmark = pytest.mark.gpu

TOL_FP32 = 1e-4     # max|a-b| / max|b| per row, float32 configuration
TOL_BF16 = 2e-2     # bf16 configurations
TIE_GAP = 1e-2      # token mismatches are allowed only where the oracle's top-2 gap is below this

SMALL_BF16 = get_config("c0", name="small_bf16", n_layers=3, d_model=256, n_heads=4, n_kv_heads=2, head_dim=64,
                        d_ffn=704, vocab=3000, dtype="bf16", seed=21, norm_gain="random", rope_base=1e6)
SMALL_BF16_D128 = SMALL_BF16.with_(name="small_bf16_d128", n_heads=2, n_kv_heads=2, head_dim=128, n_medusa=4,
                                   topk=(10, 4, 2, 2), tree_nodes=64, seed=22, vocab=32016)


@pytest.fixture(scope="module")
def torch():
    t = pytest.importorskip("torch")
    if not t.cuda.is_available():
        pytest.skip("no CUDA device")
    return t


def _lockstep(cfg, tol, new_tokens, prompt_len=None, tree_nodes=None, flags=0, **kw):
    from paper_2503_14153_b200 import build_tree
    from tests_lockstep import run_lockstep
    w = draw_weights(cfg)
    prompt = draw_prompt(cfg, prompt_len)
    tree = build_tree(cfg.topk, tree_nodes or cfg.tree_nodes)
    return run_lockstep(cfg, w, tree, prompt, new_tokens, tol, TIE_GAP, flags=flags, **kw)


def test_c0_tiny_fp32_full_run(torch):
    """Configuration 0 end to end: 32-token prompt, 16-node tree, 64 new tokens, float32."""
    cfg = get_config("c0")
    rep = _lockstep(cfg, TOL_FP32, cfg.new_tokens, check_kv_every=8)
    assert len(rep.tokens) >= cfg.new_tokens
    assert not rep.near_ties, rep.near_ties
    assert rep.max_logit_err < TOL_FP32 and rep.max_kv_err < TOL_FP32


def test_c0_chain_tree_and_single_node_tree(torch):
    from paper_2503_14153_b200 import chain_tree
    from tests_lockstep import run_lockstep
    cfg = get_config("c0")
    w, prompt = draw_weights(cfg), draw_prompt(cfg)
    a = run_lockstep(cfg, w, chain_tree(cfg.n_medusa + 1), prompt, 24, TOL_FP32)
    b = run_lockstep(cfg, w, chain_tree(1), prompt, 24, TOL_FP32)
    assert a.tokens[:24] == b.tokens[:24]
    assert b.counts == [1] * len(b.counts)


def test_c0_random_gains_and_ragged_prompt(torch):
    cfg = get_config("c0", norm_gain="random", seed=5)
    rep = _lockstep(cfg, TOL_FP32, 20, prompt_len=37, tree_nodes=11)
    assert rep.steps > 0


def test_c0_long_prompt_spans_several_prefill_passes(torch):
    cfg = get_config("c0", seed=6)
    rep = _lockstep(cfg, TOL_FP32, 12, prompt_len=300, check_kv_every=4)
    assert rep.max_kv_err < TOL_FP32


def test_small_bf16_simple_kernels(torch):
    from paper_2503_14153_b200 import FLAG_SIMPLE_KERNELS
    rep = _lockstep(SMALL_BF16, TOL_BF16, 24, prompt_len=45, flags=FLAG_SIMPLE_KERNELS, check_kv_every=6)
    assert rep.max_logit_err < TOL_BF16


def test_small_bf16_tensor_core_path(torch):
    rep = _lockstep(SMALL_BF16, TOL_BF16, 32, prompt_len=45, check_kv_every=6)
    assert rep.max_logit_err < TOL_BF16


def test_small_bf16_d128_tree64_tensor_core_path(torch):
    rep = _lockstep(SMALL_BF16_D128, TOL_BF16, 24, prompt_len=150, check_kv_every=6)
    assert rep.max_logit_err < TOL_BF16


def test_small_bf16_d512_cluster_epilogues(torch):
    """A width at which every projection with a cluster epilogue takes it (output projection K = 512 = 8
    chunks for the 8-CTA cluster; gate+up as clusters of 3 with the SwiGLU inside; down projection
    K = 1344; q/k/v with RoPE and the cache store inside), with a d_ffn that leaves the last tile half empty,
    against the oracle: all cluster epilogues on, the default set, none, and smaller trees."""
    from paper_2503_14153_b200 import SpecDecoder, build_tree, upload_weights
    from paper_2503_14153_b200 import binding as B
    from tests_lockstep import run_lockstep
    cfg = SMALL_BF16.with_(name="small_bf16_d512", d_model=512, n_heads=4, n_kv_heads=4, head_dim=128, d_ffn=1344,
                           n_medusa=4, topk=(10, 4, 2, 2), tree_nodes=64, seed=24)
    w, prompt = draw_weights(cfg), draw_prompt(cfg, 150)
    tree = build_tree(cfg.topk, cfg.tree_nodes)
    dw = upload_weights(cfg, w)
    for mask in (7, 2, 0):        # every cluster epilogue; the default (gate+up only); none
        gpu = SpecDecoder(cfg, dw, tree, 150 + 24 + 8, flags=B.FLAG_KEEP_LOGITS)
        gpu.set_option(B.OPT_CLUSTER_EPILOGUE, mask)
        rep = run_lockstep(cfg, w, tree, prompt, 24, TOL_BF16, TIE_GAP, check_kv_every=3, gpu=gpu)
        gpu.close()
        assert rep.steps > 0
    for T in (16, 32):
        gpu = SpecDecoder(cfg, dw, build_tree(cfg.topk, T), 40 + 8 + 8, flags=B.FLAG_KEEP_LOGITS)
        gpu.set_option(B.OPT_CLUSTER_EPILOGUE, 7)
        r2 = run_lockstep(cfg, w, build_tree(cfg.topk, T), prompt[:40], 8, TOL_BF16, TIE_GAP, gpu=gpu)
        gpu.close()
        assert r2.steps > 0


@pytest.mark.parametrize("T,prompt_len,umma", [(64, 70, 1), (64, 700, 1), (128, 300, 1), (16, 150, 1), (32, 1100, 1),
                                                (64, 700, 0), (128, 300, 0)])
def test_long_context_attention_kernels_on_small_shapes(torch, T, prompt_len, umma):
    """The long-context attention kernels (tcgen05 scores and P V with umma = 1, the shared-K/V mma.sync kernel with
    umma = 0) forced onto short contexts by lowering their threshold to one position: one and several 128-key
    tiles, key splits merged inside a cluster (umma = 1) or by the last CTA (umma = 0), idle splits, two row halves at T = 128, trees of 16 and 32 rows, and prompt
    processing in 128-row passes, all against the oracle."""
    from paper_2503_14153_b200 import SpecDecoder, build_tree, upload_weights
    from paper_2503_14153_b200 import binding as B
    from tests_lockstep import run_lockstep
    cfg = SMALL_BF16_D128.with_(tree_nodes=T, seed=25)
    w, prompt = draw_weights(cfg), draw_prompt(cfg, prompt_len)
    tree = build_tree(cfg.topk, T)
    gpu = SpecDecoder(cfg, upload_weights(cfg, w), tree, prompt_len + 40, flags=B.FLAG_KEEP_LOGITS)
    gpu.set_option(B.OPT_ATTN_UMMA, umma)
    gpu.set_option(B.OPT_LONG_ATTN_KEYS, 1)
    rep = run_lockstep(cfg, w, tree, prompt, 12, TOL_BF16, TIE_GAP, gpu=gpu, check_kv_every=4)
    gpu.close()
    assert rep.steps > 0


@pytest.mark.parametrize("umma,wide", [(1, 1), (0, 1), (1, 0)])
def test_long_context_attention_kernels_batched_ragged(torch, umma, wide):
    """The long-context attention kernels on a batch of four ragged sequences (17 to 530 cached positions: less
    than one 128-key tile up to several tiles with a ragged tail; sequence b's pages interleave with the others'
    in the pool), every sequence in lock step with an oracle of its own for three steps. The passes have 256 rows
    (512 in the prompt): the projections run as 128 x 256 tiles (wide = 1) or on the weight streamer (wide = 0),
    and the glue kernels take their many-row forms on finished sums or on partial sums."""
    from oracle.decoder import OracleModel
    from oracle.spec import OracleSpecDecoder
    from paper_2503_14153_b200 import SpecDecoder, build_tree, upload_weights
    from paper_2503_14153_b200 import binding as B
    from tests_lockstep import run_lockstep_batch
    cfg = SMALL_BF16_D128.with_(tree_nodes=64, seed=27)
    w = draw_weights(cfg)
    lengths = (17, 530, 129, 256)
    prompts = [draw_prompt(cfg.with_(seed=27 + i), n) for i, n in enumerate(lengths)]
    tree = build_tree(cfg.topk, 64)
    model = OracleModel(cfg, w)
    gpu = SpecDecoder(cfg, upload_weights(cfg, w), tree, 530 + 40, max_batch=4, flags=B.FLAG_KEEP_LOGITS)
    gpu.set_option(B.OPT_ATTN_UMMA, umma)
    gpu.set_option(B.OPT_WIDE_GEMM, wide)
    gpu.set_option(B.OPT_LONG_ATTN_KEYS, 1)
    oracles = {b: OracleSpecDecoder(model, tree, 530 + 40) for b in range(4)}
    reps = run_lockstep_batch(cfg, gpu, oracles, prompts, 3, TOL_BF16, TIE_GAP)
    gpu.close()
    for b, rep in reps.items():
        assert rep.steps == 3, b


def test_ten_heads_deep_tree(torch):
    """The paper's head count (K = 10): ten stacked head matrices (three GEMM launches), a tree ten levels deep."""
    cfg = SMALL_BF16.with_(name="small_bf16_k10", n_medusa=10, topk=(4, 3, 2, 2, 2, 1, 1, 1, 1, 1), tree_nodes=48, seed=23)
    rep = _lockstep(cfg, TOL_BF16, 16, prompt_len=40)
    assert rep.max_logit_err < TOL_BF16


def test_controlled_draft_accept_lengths(torch):
    """Controlled-acceptance draft: rank-0 candidate of head j is the true greedy token with
    probability p. The stream is unchanged and the accepted lengths match the oracle's."""
    from oracle.decoder import OracleModel
    from oracle.spec import OracleSpecDecoder
    from oracle.tree import chain_tree as o_chain
    cfg = SMALL_BF16
    w, prompt = draw_weights(cfg), draw_prompt(cfg, 20)
    model = OracleModel(cfg, w)
    stream = OracleSpecDecoder(model, o_chain(1), 200).generate(prompt, 80)[0]
    uniforms, hit = controlled_draft(cfg, stream, 0.7, 80)

    def ov(i, done):
        t = uniforms[i, :, :].copy()
        for j in range(cfg.n_medusa):
            if hit[i, j] and done + 1 + j < len(stream):
                t[j, 0] = stream[done + 1 + j]
        return t

    from paper_2503_14153_b200 import build_tree
    from tests_lockstep import run_lockstep
    tree = build_tree(cfg.topk, cfg.tree_nodes)
    rep = run_lockstep(cfg, w, tree, prompt, 60, TOL_BF16, overrides=lambda i, done: ov(i, done)[:, :max(cfg.topk)],
                       oracle_model=model)
    ties = {t[0] for t in rep.near_ties}
    if not ties:
        assert rep.tokens[:60] == [int(t) for t in stream[:60]]
    assert np.mean(rep.counts) > 1.5


def test_fragment_truncation(torch):
    from oracle.decoder import OracleModel
    from oracle.spec import OracleSpecDecoder
    from oracle.tree import chain_tree as o_chain
    cfg = get_config("c0")
    w, prompt = draw_weights(cfg), draw_prompt(cfg)
    stream = OracleSpecDecoder(OracleModel(cfg, w), o_chain(1), 200).generate(prompt, 40)[0]
    frag = int(np.bincount(stream).argmax())
    rep = _lockstep(cfg, TOL_FP32, 40, frag_token=frag)
    assert rep.tokens[:40] == [int(t) for t in stream[:40]]


def test_typical_acceptance_mode(torch):
    cfg = get_config("c0")
    rep = _lockstep(cfg, TOL_FP32, 30, accept_mode=1, typ=(0.3, 0.6, 1.0))
    assert rep.steps > 0


@pytest.mark.parametrize("temperature", [0.5, 2.0])
def test_typical_acceptance_at_a_temperature(torch, temperature):
    """Eq. 1 with p = softmax(logits / temperature), temperature != 1, argmax next token."""
    cfg = get_config("c0")
    rep = _lockstep(cfg, TOL_FP32, 30, accept_mode=1, typ=(0.3, 0.6, temperature))
    assert rep.steps > 0 and max(rep.counts) > 1


@pytest.mark.parametrize("seed", [7, (5 << 32) + 11])
def test_sampled_decoding_temperature_0p8(torch, seed):
    """Sampled decoding at temperature 0.8 (Sec. IV-B times every prompt greedy and sampled): Eq. 1
    acceptance and the next token drawn at the step's Philox uniform, token for token against the
    oracle (both sides draw the same uniforms; a draw may differ only at a boundary of the
    cumulative distribution)."""
    cfg = get_config("c0")
    t = float(np.float32(0.8))          # the value the float32 field of the configuration holds
    rep = _lockstep(cfg, TOL_FP32, 48, accept_mode=1, typ=(0.09, 0.3, t), sampling=True, seed=seed)
    assert rep.steps > 0 and len(rep.near_ties) <= 1
    greedy = _lockstep(cfg, TOL_FP32, 48, accept_mode=1, typ=(0.09, 0.3, t))
    assert rep.tokens != greedy.tokens          # the draws matter: not the argmax stream
    other = _lockstep(cfg, TOL_FP32, 16, accept_mode=1, typ=(0.09, 0.3, t), sampling=True, seed=seed + 1)
    assert other.tokens[:16] != rep.tokens[:16]


@pytest.mark.parametrize("M,N,K,ctas", [(16, 128, 64, 1), (64, 384, 256, 2), (64, 4096, 4096, 296),
                                        (128, 1000, 704, 7), (32, 200, 128, 3), (256, 512, 512, 148),
                                        (64, 12288, 4096, 296), (48, 1000, 1408, 37)])
def test_op_linear_bf16_vs_oracle_matmul(torch, M, N, K, ctas):
    from oracle.numerics import round_bf16
    from paper_2503_14153_b200 import spec_op_linear
    rng = np.random.default_rng(M * 7 + N)
    x = round_bf16(rng.standard_normal((M, K)).astype(np.float32))
    w = round_bf16((rng.standard_normal((N, K)) * 0.05).astype(np.float32))
    ref = x @ w.T
    y = spec_op_linear(torch.from_numpy(x.astype(np.float32)).cuda().to(torch.bfloat16),
                       torch.from_numpy(w.astype(np.float32)).cuda().to(torch.bfloat16), ctas).cpu().numpy()
    err = np.abs(y - ref).max() / np.abs(ref).max()
    assert err < 1e-5, err


def test_op_linear_fp32_vs_oracle_matmul(torch):
    from paper_2503_14153_b200 import spec_op_linear
    rng = np.random.default_rng(3)
    x, w = rng.standard_normal((13, 688)).astype(np.float32), rng.standard_normal((301, 688)).astype(np.float32)
    y = spec_op_linear(torch.from_numpy(x).cuda(), torch.from_numpy(w).cuda()).cpu().numpy()
    ref = x.astype(np.float64) @ w.astype(np.float64).T
    assert np.abs(y - ref).max() / np.abs(ref).max() < 1e-5


@pytest.mark.parametrize("n_seq,seq_len,K", [(1, 10, 3), (3, 8192, 10), (2, 257, 4), (1, 1, 10), (5, 1000, 0), (0, 16, 3)])
def test_build_labels_vs_oracle(torch, n_seq, seq_len, K):
    """Syntax-enriched labels (Sec. III-C): bit-exact against the oracle, ragged tails and empty input included."""
    from oracle.labels import syntax_enriched_labels
    from paper_2503_14153_b200 import spec_build_labels
    frag, pad, ign = 32016, 32017, -100
    rng = np.random.default_rng(seq_len * 31 + K)
    toks = rng.integers(0, 32016, size=(n_seq, seq_len)).astype(np.int32)
    toks[rng.random(toks.shape) < 0.15] = frag
    got = spec_build_labels(torch.from_numpy(toks).cuda(), K, frag, pad, ign).cpu().numpy()
    assert got.shape == (n_seq, K + 1, seq_len)
    for i in range(n_seq):
        assert np.array_equal(got[i], syntax_enriched_labels(toks[i], K, frag, pad, ign))


def test_error_returns_and_degenerate_shapes(torch):
    """Calls out of order and sequences that run out of room return error codes (nothing faults); a
    one-token prompt and a model without extra heads (every step emits exactly the root) still decode."""
    from paper_2503_14153_b200 import SpecDecoder, SpecError, build_tree, chain_tree, upload_weights
    from tests_lockstep import run_lockstep
    cfg = get_config("c0")
    w = draw_weights(cfg)
    dw = upload_weights(cfg, w)
    tree = build_tree(cfg.topk, cfg.tree_nodes)
    dec = SpecDecoder(cfg, dw, tree, max_seq=40)
    with pytest.raises(SpecError) as e:
        dec.step()
    assert e.value.code == -7                      # step before prefill
    with pytest.raises(SpecError) as e:
        dec.prefill(draw_prompt(cfg, 39))          # leaves no room to generate within max_seq
    assert e.value.code == -4
    dec.prefill(draw_prompt(cfg, 30))
    with pytest.raises(SpecError) as e:
        for _ in range(20):
            dec.step()
    assert e.value.code == -4                      # ran into max_seq after a few steps
    dec.close()
    # one-token prompt
    rep = run_lockstep(cfg, w, tree, draw_prompt(cfg, 1), 8, TOL_FP32)
    assert rep.steps > 0
    # no extra heads: the tree is the root alone
    cfg0 = get_config("c0", n_medusa=0, topk=(), tree_nodes=1)
    w0 = draw_weights(cfg0)
    dec = SpecDecoder(cfg0, upload_weights(cfg0, w0), chain_tree(1), max_seq=64)
    dec.prefill(draw_prompt(cfg0, 9))
    for _ in range(3):
        tok, cnt = dec.step()
        assert int(cnt[0]) == 1
    dec.close()


def test_bounded_wait_times_out_and_context_survives(torch):
    """A device-side wait that nothing completes gives up after its limit: the library reports
    SPEC_E_TIMEOUT with the place code, and the same context decodes on afterwards."""
    from paper_2503_14153_b200 import SpecDecoder, build_tree, upload_weights
    cfg = get_config("c0")
    w = draw_weights(cfg)
    dec = SpecDecoder(cfg, upload_weights(cfg, w), build_tree(cfg.topk, cfg.tree_nodes), max_seq=96)
    prompt = draw_prompt(cfg)
    dec.prefill(prompt)
    tok0, cnt0 = dec.step()
    assert dec.wait_timeout_probe(1000) == -6                 # SPEC_E_TIMEOUT after 1 ms
    msg = dec.lib.spec_last_error(dec._ctx).decode()
    assert "status 1 at 99" in msg, msg
    assert dec.wait_timeout_probe(0) == -1                    # limit out of range: refused, nothing launched
    assert dec.debug(5 + 5)[0] == 0                           # status word is clean again (SPEC_DBG_STATUS)
    tok1, cnt1 = dec.step()                                   # the context is still usable
    assert 1 <= int(cnt1[0]) <= cfg.n_medusa + 1
    # and the stream is what an undisturbed decoder emits
    ref = SpecDecoder(cfg, upload_weights(cfg, w), build_tree(cfg.topk, cfg.tree_nodes), max_seq=96)
    ref.prefill(prompt)
    a, ca = ref.step()
    b, cb = ref.step()
    assert list(a[0][:int(ca[0])]) == list(tok0[0][:int(cnt0[0])]) and list(b[0][:int(cb[0])]) == list(tok1[0][:int(cnt1[0])])
    dec.close(); ref.close()


def test_timeline_and_options(torch):
    """The device timeline lists every launch of a step in order with start <= end; tuning knobs
    reject out-of-range values and do not change the emitted tokens."""
    from paper_2503_14153_b200 import SpecDecoder, SpecError, build_tree, upload_weights
    from paper_2503_14153_b200 import binding as B
    cfg = SMALL_BF16
    w = draw_weights(cfg)
    dw = upload_weights(cfg, w)
    tree = build_tree(cfg.topk, cfg.tree_nodes)
    prompt = draw_prompt(cfg, 33)

    def run(opts):
        dec = SpecDecoder(cfg, dw, tree, 200)
        for k, v in opts.items():
            dec.set_option(k, v)
        dec.prefill(prompt)
        out = []
        for _ in range(6):
            tok, cnt = dec.step()
            out.extend(int(t) for t in tok[0][: int(cnt[0])])
        return dec, out

    dec, base = run({})
    with pytest.raises(SpecError):
        dec.set_option(B.OPT_GEMM_CTAS, 0)
    with pytest.raises(SpecError):
        dec.set_option(99, 1)
    with pytest.raises(SpecError):
        dec.trace()                                     # tracing is off
    with pytest.raises(SpecError):
        dec.phase_ms()                                  # phase timing is off
    dec.set_option(B.OPT_PHASE_TIMING, 1)
    dec.step()
    ph = dec.phase_ms()
    assert ph.shape == (5,) and (ph > 0).all() and ph[2] == ph.max()   # the verification forward dominates
    dec.set_option(B.OPT_PHASE_TIMING, 0)
    dec.set_option(B.OPT_TRACE, 1)
    l0 = dec.query(B.Q_KERNEL_LAUNCHES)
    dec.step()
    n_launch = dec.query(B.Q_KERNEL_LAUNCHES) - l0
    tr = dec.trace()
    assert len(tr) == n_launch and n_launch > 10
    names = [r[0] for r in tr]
    assert names[-1] == "compact_kv" and "attention_tc" in names and any(n.startswith("gemm") for n in names)
    for name, t0, t1, _, _ in tr:
        assert 0 < t0 <= t1, (name, t0, t1)
    assert tr[0][1] <= tr[-1][2]
    dec.close()
    # programmatic dependent launch and L2 prefetch never change results; the CTA count only the
    # summation order (same tokens here: no near-tie in these steps)
    for opts in ({B.OPT_PDL: 0}, {B.OPT_L2_PREFETCH: 4}, {B.OPT_GRAPH: 0}):
        d2, out = run(opts)
        d2.close()
        assert out == base


def test_step_graph_replay(torch):
    """The step is recorded into a CUDA graph once and replayed: one recording serves the steps until a
    sequence passes the 768-position bound of the single-split attention launch, then one more is made
    (for every longer length); a new prefill and an option change also start a new recording; the
    tokens are those of direct enqueue."""
    from paper_2503_14153_b200 import SpecDecoder, build_tree, upload_weights
    from paper_2503_14153_b200 import binding as B
    cfg = SMALL_BF16
    dw = upload_weights(cfg, draw_weights(cfg))
    tree = build_tree(cfg.topk, cfg.tree_nodes)
    prompt = draw_prompt(cfg, 700)

    def run(graph, steps):
        dec = SpecDecoder(cfg, dw, tree, 1100)
        dec.set_option(B.OPT_GRAPH, graph)
        dec.prefill(prompt)
        out, caps = [], []
        for _ in range(steps):
            tok, cnt = dec.step()
            out.extend(int(t) for t in tok[0][: int(cnt[0])])
            caps.append(dec.query(B.Q_GRAPH_CAPTURES))
        return dec, out, caps

    d0, direct, caps0 = run(0, 60)
    assert caps0[-1] == 0
    d0.close()
    d1, replay, caps1 = run(1, 60)
    assert replay == direct
    # 700 prompt tokens + 16 tree rows fit the 768-position bound for the first steps only
    assert caps1[0] == 1 and caps1[5] == 1 and caps1[-1] == 2, caps1
    launches = d1.query(B.Q_KERNEL_LAUNCHES)
    d1.step()
    assert d1.query(B.Q_KERNEL_LAUNCHES) - launches > 10        # replayed launches are counted
    d1.set_option(B.OPT_PDL, 0)
    d1.step()
    assert d1.query(B.Q_GRAPH_CAPTURES) == 3
    d1.prefill(prompt)
    d1.step()
    assert d1.query(B.Q_GRAPH_CAPTURES) == 4
    d1.close()


def test_packed_weight_image_and_equivalence(torch):
    """spec_pack_weight writes, unit by unit, the shared-memory image a swizzled TMA load of the tile
    leaves (checked against a NumPy construction of that layout, ragged last tile zero-filled); a
    decoder on pre-tiled weights emits bit-identical results to one on the row-major matrices."""
    from paper_2503_14153_b200 import SpecDecoder, build_tree, upload_weights, spec_pack_weight
    from paper_2503_14153_b200 import binding as B
    rows, cols = 300, 192
    rng = np.random.default_rng(5)
    w = torch.from_numpy(rng.standard_normal((rows, cols)).astype(np.float32)).cuda().bfloat16().contiguous()
    img = spec_pack_weight(w).cpu().numpy().view(np.uint16)
    src = w.view(torch.int16).cpu().numpy().view(np.uint16)
    tiles, KC = (rows + 127) // 128, cols // 64
    want = np.zeros((tiles, KC, 128, 8, 8), dtype=np.uint16)          # [tile][kc][row][chunk position][8 elements]
    for t in range(tiles):
        for kc in range(KC):
            for r in range(128):
                if t * 128 + r < rows:
                    for ch in range(8):
                        want[t, kc, r, ch ^ (r & 7)] = src[t * 128 + r, kc * 64 + ch * 8: kc * 64 + ch * 8 + 8]
    assert img.size == want.size and np.array_equal(img, want.reshape(-1))

    cfg = SMALL_BF16_D128
    dw = upload_weights(cfg, draw_weights(cfg))
    tree = build_tree(cfg.topk, cfg.tree_nodes)
    prompt = draw_prompt(cfg, 90)
    outs = []
    for packed in (True, False):
        dec = SpecDecoder(cfg, dw, tree, 300, flags=B.FLAG_KEEP_LOGITS, packed=packed)
        assert dec.packed == packed
        dec.prefill(prompt)
        toks = []
        for _ in range(5):
            tok, cnt = dec.step()
            toks.extend(int(x) for x in tok[0][: int(cnt[0])])
        outs.append((toks, dec.debug(B.DBG_LOGITS).copy(), dec.debug(B.DBG_HIDDEN).copy()))
        dec.close()
    assert outs[0][0] == outs[1][0]
    assert np.array_equal(outs[0][1], outs[1][1]) and np.array_equal(outs[0][2], outs[1][2])
