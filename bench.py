#!/usr/bin/env python
"""Benchmark of the draft-and-verify decode loop on the CodeLlama-7B shape (configuration 1).

One "step" is one spec_step: extra heads + top-k, tree expansion, tree-masked verification
forward, acceptance, KV compaction. `value` is decode tokens/s with everything resident in HBM
and steps enqueued back to back; `e2e` is the same loop through the C ABI with host buffers
(candidate override table copied in, emitted tokens copied out, every step).
"""
import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
for p in (ROOT,):
    if p not in sys.path:
        sys.path.insert(0, p)

METRIC = "decode tokens/sec at batch 1 (7B shape)"
UNIT = "tokens/s"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu, self.proc, self.path = gpu_index, None, None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for line in open(self.path):
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        os.unlink(self.path)
        if sm:
            out = {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                   "samples": len(sm)}
        return out


def aggregate_replicas(seconds: float, units: float, world: int, device="cpu"):
    """Whole-job figures of `world` independent replicas: the slowest rank's time (max) and all ranks'
    units (sum). With world > 1 the default process group must be initialised."""
    import torch
    t = torch.tensor([seconds], dtype=torch.float64, device=device)
    u = torch.tensor([float(units)], dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def algorithmic_bytes(cfg, n_ctx: int, T: int):
    """Bytes one step must read: verify = layer weights + lm_head + cached K/V + tree activations;
    the whole step adds the head matrices and the heads' pass over lm_head."""
    e = 2 if cfg.dtype == "bf16" else 4
    d, F, V = cfg.d_model, cfg.d_ffn, cfg.vocab
    HD, KD = cfg.n_heads * cfg.head_dim, cfg.n_kv_heads * cfg.head_dim
    layer = d * HD + 2 * d * KD + HD * d + 3 * d * F
    verify = e * (cfg.n_layers * layer + V * d) + n_ctx * 2 * cfg.n_layers * KD * e + T * d * e
    step = verify + e * (cfg.n_medusa * (d * d + d) + V * d)
    gate_up = e * (2 * F * d) + T * d * e + T * F * e
    return verify, step, gate_up


def oracle_step_sample(cfg, weights_host, tree, prompt_len=16, layers=None):
    """Times the CPU oracle: one draft-and-verify step after a short prompt. Returns
    (seconds per step, tokens emitted, threads used)."""
    from oracle.decoder import OracleModel
    from oracle.spec import OracleSpecDecoder
    from synthetic import draw_prompt
    ocfg = cfg if layers is None else cfg.with_(n_layers=layers)
    model = OracleModel(ocfg, weights_host)
    dec = OracleSpecDecoder(model, tree, prompt_len + 64)
    dec.prefill(draw_prompt(cfg, prompt_len))
    t0 = time.perf_counter()
    rec = dec.step()
    dt = time.perf_counter() - t0
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        threads = os.cpu_count() or 1
    return dt, int(rec["count"]), threads


def run_reference(args, rank):
    """The reference arm: the CPU oracle as it stands, timed on the host cores."""
    if rank != 0:
        return
    from paper_2503_14153_b200 import build_tree
    from synthetic import draw_tensor, get_config, tensor_specs
    cfg = get_config(args.config)
    tree = build_tree(cfg.topk, cfg.tree_nodes)
    total = args.steps + args.warmup
    layers = 1 if total > 12 else (4 if total > 3 else cfg.n_layers)
    ocfg = cfg.with_(n_layers=layers)
    w = {}
    for idx, (name, shape, kind) in enumerate(tensor_specs(cfg)):
        if name.startswith("layers.") and int(name.split(".")[1]) >= layers:
            continue
        w[name] = draw_tensor(cfg, idx, shape, kind)
    from oracle.decoder import OracleModel
    from oracle.spec import OracleSpecDecoder
    from synthetic import draw_prompt
    dec = OracleSpecDecoder(OracleModel(ocfg, w), tree, 16 + (total + 2) * (cfg.n_medusa + 1) + 64)
    dec.prefill(draw_prompt(cfg, 16))
    # split of a step: heads + lm_head do not scale with depth, the layer stack does
    times, toks = [], 0
    t_budget = time.perf_counter()
    for i in range(total):
        t0 = time.perf_counter()
        rec = dec.step()
        dt = time.perf_counter() - t0
        if i >= args.warmup:
            times.append(dt); toks += int(rec["count"])
        if time.perf_counter() - t_budget > 240 and len(times) >= 1:
            break
    # time of the part that does not scale with depth: one candidates() call + one lm_head product
    t0 = time.perf_counter(); dec.candidates(); t_heads = time.perf_counter() - t0
    from oracle.decoder import medusa_logits  # noqa: F401
    hq = np.zeros((cfg.tree_nodes, cfg.d_model))
    t0 = time.perf_counter(); _ = hq @ w["lm_head"].astype(np.float64).T; t_lm = time.perf_counter() - t0
    mean_sample = float(np.mean(times))
    fixed = min(t_heads + t_lm, mean_sample * 0.9)
    full_step = fixed + (mean_sample - fixed) * cfg.n_layers / layers
    steps_done = len(times)
    value = (toks / steps_done) / full_step
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        threads = os.cpu_count() or 1
    sample = (f"oracle draft-and-verify steps (T={cfg.tree_nodes}, 16-token prompt) on the first {layers} of "
              f"{cfg.n_layers} layers; layer-stack time scaled by {cfg.n_layers}/{layers}, heads+lm_head time kept; "
              f"{steps_done} timed steps")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps_done, "warmup": args.warmup, "ms_per_step": full_step * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "tree_nodes": cfg.tree_nodes, "prompt_len": 16, "batch": 1},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="c1")
    ap.add_argument("--layers", type=int, default=None, help="override the layer count (profiling of small cases)")
    ap.add_argument("--prompt-len", type=int, default=None)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the e2e, per-kernel and CPU legs (profiling)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    import torch.distributed as dist
    from paper_2503_14153_b200 import SpecDecoder, build_tree, load_library
    from paper_2503_14153_b200 import binding as B
    from synthetic import draw_prompt, get_config, stream_weights_to_device
    load_library()   # fails loudly when the CUDA extension is missing
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))

    cfg = get_config(args.config)
    if args.layers:
        cfg = cfg.with_(n_layers=args.layers)
    if args.prompt_len:
        cfg = cfg.with_(prompt_len=args.prompt_len)
    tree = build_tree(cfg.topk, cfg.tree_nodes)
    K, T = cfg.n_medusa, cfg.tree_nodes
    want_cpu = rank == 0 and world == 1 and not args.no_cpu_baseline and not args.no_extras
    host_w = {} if want_cpu else None
    t0 = time.time()
    dw = stream_weights_to_device(cfg, dev, threads=min(16, os.cpu_count() or 8), keep_host=host_w)
    t_weights = time.time() - t0
    total_steps = (args.warmup + args.steps) * 2 + 64
    max_seq = cfg.prompt_len + total_steps * (K + 1) + 16
    dec = SpecDecoder(cfg, dw, tree, max_seq)
    prompt = draw_prompt(cfg)
    peak, peak_kind = measured_peaks()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    # ---------------- device-resident loop: steps enqueued back to back ----------------
    dec.prefill(prompt)
    for _ in range(args.warmup):
        dec.step_async()
    n_before = len(dec.read_generated(0))
    launches0 = dec.query(B.Q_KERNEL_LAUNCHES)
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    stream = torch.cuda.current_stream()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record(stream)
    for _ in range(args.steps):
        dec.step_async()
    ev1.record(stream)
    barrier()
    ms = ev0.elapsed_time(ev1)
    clocks = sampler.stop()
    launches = dec.query(B.Q_KERNEL_LAUNCHES) - launches0
    gen = dec.read_generated(0)
    tokens = len(gen) - n_before
    n_ctx_mid = cfg.prompt_len + n_before + tokens // 2
    # the phase boundaries of one more step, outside the timed region (the events cost overlap)
    dec.set_option(B.OPT_PHASE_TIMING, 1)
    dec.step_async()
    phase = dec.phase_ms()
    dec.set_option(B.OPT_PHASE_TIMING, 0)
    ms_max, tokens_all = aggregate_replicas(ms, tokens, world, dev)
    value = tokens_all / (ms_max * 1e-3)
    ms_per_step = ms_max / args.steps

    verify_b, step_b, gate_up_b = algorithmic_bytes(cfg, n_ctx_mid, T)
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": cfg.dtype, "data": "synthetic",
        "config": {"workload": cfg.name, "layers": cfg.n_layers, "d_model": cfg.d_model, "tree_nodes": T,
                   "medusa_heads": K, "prompt_len": cfg.prompt_len, "batch": 1, "page_size": cfg.page_size,
                   "weight_layout": "pre-tiled (spec_pack_weight)" if dec.packed else "row-major",
                   "parallelism": "replicas" if world > 1 else "single",
                   "l2": "weights streamed per step (13.6 GB) exceed the 126 MB L2; no flush needed"},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "mean_accepted_len": tokens / args.steps,
        "spec_step_us": ms_per_step * 1e3,
        "verify_step_us_last": float(phase[2]) * 1e3,
        "phase_us_last": {k: float(v) * 1e3 for k, v in zip(("heads", "expand", "verify", "accept", "compact"), phase)},
        "step_hbm": {"algorithmic_bytes": step_b, "achieved_gbs": step_b / (ms_per_step * 1e-3) / 1e9,
                     "frac_of_measured_peak": step_b / (ms_per_step * 1e-3) / 1e9 / peak, "peak_gbs": peak,
                     "peak_kind": peak_kind, "frac_of_8tbs": step_b / (ms_per_step * 1e-3) / 8e12},
        "weights_setup_s": t_weights,
    }

    if not args.no_extras:
        # ---------------- end to end through the C ABI with host buffers ----------------
        dec.prefill(prompt)
        keep = np.full((1, K, dec.kmax), -1, dtype=np.int32)
        for _ in range(args.warmup):
            dec.step(keep)
        barrier()
        t0 = time.perf_counter()
        e_tokens = 0
        for _ in range(args.steps):
            _, cnt = dec.step(keep)
            e_tokens += int(cnt[0])
        torch.cuda.synchronize()
        e_s = time.perf_counter() - t0
        e_max, e_tok_all = aggregate_replicas(e_s, e_tokens, world, dev)
        out["e2e"] = {"value": e_tok_all / e_max, "unit": UNIT,
                      "h2d_bytes_per_step": int(keep.nbytes), "d2h_bytes_per_step": int((K + 1) * 4 + 4 + 4 + 16),
                      "ms_per_step": e_max * 1e3 / args.steps}

        # ---------------- dominant kernel: gate/up projection with fused SwiGLU ----------------
        dec.profile_kernel(B.PROFILE_GATE_UP)
        for _ in range(min(args.steps, 20)):
            dec.step_async()
        k_ms, k_n = dec.profile_read()
        dec.profile_kernel(B.PROFILE_OFF)
        if k_n > 0:
            per = k_ms / k_n * 1e-3
            out["roofline"] = {"bound": "hbm", "kernel": "gemm_stream<64> on the gate+up projection (2 x [11008,4096] bf16 weights, pre-tiled, streamed once)",
                               "achieved": gate_up_b / per / 1e9, "peak": peak, "unit": "GB/s",
                               "frac": gate_up_b / per / 1e9 / peak,
                               # dram__bytes_read.sum + dram__bytes_write.sum of this kernel at this shape
                               # (profiles/gemm_stream_7b_shapes_ncu_full.md); null for other shapes
                               "traffic": 186.5e6 if (cfg.d_model, cfg.d_ffn, T) == (4096, 11008, 64) else None,
                               "peak_kind": peak_kind,
                               "launches_timed": int(k_n), "us_per_launch": per * 1e6,
                               "algorithmic_bytes_per_launch": gate_up_b}
        per_kernel = {}
        for name, kind in (("qkv", B.PROFILE_QKV), ("wo", B.PROFILE_WO), ("down", B.PROFILE_DOWN),
                           ("attention", B.PROFILE_ATTENTION)):
            dec.profile_kernel(kind)
            for _ in range(5):
                dec.step_async()
            k_ms, k_n = dec.profile_read()
            per_kernel[name] = k_ms / max(k_n, 1) * 1e3
        dec.profile_kernel(B.PROFILE_OFF)
        out["kernel_us"] = per_kernel
        # device timeline of one step (GPU global timer): per kernel kind, span from first block start to
        # last block end, averaged over its launches; the GEMMs also report operands-landed -> last MMA issued
        dec.set_option(B.OPT_TRACE, 1)
        dec.step_async()
        tr = dec.trace()
        dec.set_option(B.OPT_TRACE, 0)
        agg = {}
        for name, t_start, t_end, m2, m3 in tr:
            a = agg.setdefault(name, [0, 0.0, 0.0])
            a[0] += 1
            a[1] += (t_end - t_start) / 1e3
            if name.startswith("gemm") and m2 < (1 << 62) and m3 > 0:
                a[2] += (m3 - m2) / 1e3
        out["timeline_us"] = {k: {"launches": v[0], "span_avg": round(v[1] / v[0], 2),
                                  **({"stream_window_avg": round(v[2] / v[0], 2)} if v[2] > 0 else {})} for k, v in agg.items()}
        if tr:
            out["timeline_us"]["step_span"] = round((max(r[2] for r in tr) - min(r[1] for r in tr)) / 1e3, 1)

        # ---------------- context: plain autoregressive decoding on the same kernels ----------------
        # One-node tree, no extra heads: what a token costs without speculation. The step rate of the
        # tree-verifying decoder times the accepted length Sigma_i p^i of the controlled draft (Sec. III-B
        # candidates accepted with probability p per head; the GPU tests check that the measured lengths
        # follow this form) gives the tokens/s a draft of that quality would reach on this step.
        if K > 0 and world == 1:
            from paper_2503_14153_b200 import chain_tree
            dec.close()
            cfg_ar = cfg.with_(n_medusa=0, topk=(), tree_nodes=1)
            ar = SpecDecoder(cfg_ar, dw, chain_tree(1), cfg.prompt_len + 80)
            ar.prefill(prompt)
            for _ in range(5):
                ar.step_async()
            torch.cuda.synchronize()
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a0.record(stream)
            for _ in range(40):
                ar.step_async()
            a1.record(stream)
            torch.cuda.synchronize()
            ar_ms = a0.elapsed_time(a1) / 40
            ar.close()
            out["autoregressive"] = {"ms_per_step": ar_ms, "tokens_per_s": 1e3 / ar_ms,
                                     "tree_step_over_ar_step": ms_per_step / ar_ms}
            out["tokens_per_s_at_draft_quality"] = {
                f"p={p}": {"accepted_len_closed_form": sum(p ** i for i in range(K + 1)),
                           "tokens_per_s": sum(p ** i for i in range(K + 1)) * 1e3 / ms_per_step,
                           "speedup_over_autoregressive": sum(p ** i for i in range(K + 1)) * ar_ms / ms_per_step}
                for p in (0.3, 0.6, 0.9)}

    if want_cpu:
        dt, cnt, threads = oracle_step_sample(cfg, host_w, tree)
        out["cpu_baseline"] = {"value": cnt / dt, "unit": UNIT, "cores": threads, "kind": "oracle",
                               "sample": f"1 full oracle draft-and-verify step (T={T}, all {cfg.n_layers} layers) "
                                         f"after a 16-token prompt; {dt:.1f} s"}
    dec.close()
    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
