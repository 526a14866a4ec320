"""ctypes binding of include/spec_decode.h: argument marshalling only.

PyTorch supplies device memory (weights, workspace) and the stream; every step of the
decode loop runs inside the shared library's CUDA kernels. There is no CPU fallback: if the
library is missing, loading raises.
"""
import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_NAME = "libspec_decode.so"
_lib = None

FLAG_KEEP_LOGITS = 1
FLAG_SIMPLE_KERNELS = 2
FLAG_PACKED_WEIGHTS = 4
PROFILE_OFF, PROFILE_GATE_UP, PROFILE_QKV, PROFILE_WO, PROFILE_DOWN, PROFILE_ATTENTION = range(6)

Q_KMAX, Q_KERNEL_LAUNCHES, Q_N_NODES, Q_BATCH, Q_ALGO_KIB, Q_GRAPH_CAPTURES, Q_CLUSTER_GATE_UP, Q_WIDE_GEMM = 0, 1, 2, 3, 4, 5, 6, 7
OPT_PDL, OPT_GEMM_CTAS, OPT_L2_PREFETCH, OPT_TRACE, OPT_SMALL_GEMM_CTAS, OPT_GRAPH, OPT_PHASE_TIMING, OPT_CLUSTER_EPILOGUE, OPT_WIDE_GEMM, OPT_LONG_ATTN_KEYS, OPT_ATTN_UMMA = 0, 1, 2, 3, 4, 5, 6, 7, 8, 9, 10
TRACE_NAME_LEN = 32
(DBG_TOK, DBG_POS, DBG_LOGITS, DBG_HIDDEN, DBG_ARGMAX, DBG_PATH, DBG_CAND, DBG_SEQLEN, DBG_NEXT_ROOT,
 DBG_H_LAST, DBG_STATUS) = range(11)

EXPORTS = ["spec_workspace_bytes", "spec_create", "spec_prefill", "spec_step", "spec_read_generated",
           "spec_destroy", "spec_last_error", "spec_query", "spec_debug_read", "spec_debug_read_kv",
           "spec_op_linear", "spec_op_linear_scratch_floats", "spec_op_linear_static", "spec_packed_weight_bytes",
           "spec_pack_weight", "spec_set_option", "spec_trace_read", "spec_build_labels", "spec_last_step_phase_ms", "spec_profile_kernel",
           "spec_profile_read", "spec_debug_wait_timeout"]


class SpecError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"spec error {code}: {msg}")
        self.code = code


class SpecConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab")] + \
               [("rms_eps", C.c_float), ("rope_base", C.c_float), ("dtype", C.c_int32), ("n_medusa", C.c_int32),
                ("max_batch", C.c_int32), ("max_seq", C.c_int32), ("page_size", C.c_int32), ("accept_mode", C.c_int32),
                ("typ_eps", C.c_float), ("typ_delta", C.c_float), ("temperature", C.c_float),
                ("frag_token", C.c_int32), ("flags", C.c_int32), ("sampling", C.c_int32),
                ("seed_lo", C.c_uint32), ("seed_hi", C.c_uint32)]


class SpecTree(C.Structure):
    _fields_ = [("n_nodes", C.c_int32), ("parent", C.POINTER(C.c_int32)), ("depth", C.POINTER(C.c_int32)),
                ("rank", C.POINTER(C.c_int32))]


class SpecWeights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p)] + \
               [(n, C.POINTER(C.c_void_p)) for n in ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate",
                                                     "w_up", "w_down", "medusa_w", "medusa_b")]


def library_path() -> str:
    return os.path.join(_HERE, _LIB_NAME)


def load_library():
    """Loads the CUDA shared library; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    path = library_path()
    if not os.path.exists(path):
        raise FileNotFoundError(f"{path} is missing: build it with `python -m paper_2503_14153_b200.build` "
                                "(there is no CPU fallback)")
    lib = C.CDLL(path)
    lib.spec_workspace_bytes.restype = C.c_size_t
    lib.spec_workspace_bytes.argtypes = [C.POINTER(SpecConfig), C.POINTER(SpecTree)]
    lib.spec_create.restype = C.c_int
    lib.spec_create.argtypes = [C.POINTER(SpecConfig), C.POINTER(SpecWeights), C.POINTER(SpecTree), C.c_void_p,
                                C.c_size_t, C.c_void_p, C.POINTER(C.c_void_p)]
    lib.spec_prefill.restype = C.c_int
    lib.spec_prefill.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
    lib.spec_step.restype = C.c_int
    lib.spec_step.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.spec_read_generated.restype = C.c_int
    lib.spec_read_generated.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_int32, C.POINTER(C.c_int32)]
    lib.spec_destroy.restype = C.c_int
    lib.spec_destroy.argtypes = [C.c_void_p]
    lib.spec_last_error.restype = C.c_char_p
    lib.spec_last_error.argtypes = [C.c_void_p]
    lib.spec_query.restype = C.c_int64
    lib.spec_query.argtypes = [C.c_void_p, C.c_int32]
    lib.spec_debug_read.restype = C.c_int
    lib.spec_debug_read.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_size_t]
    lib.spec_debug_read_kv.restype = C.c_int
    lib.spec_debug_read_kv.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
    lib.spec_op_linear.restype = C.c_int
    lib.spec_op_linear.argtypes = [C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32,
                                   C.c_int32, C.c_void_p, C.c_void_p]
    lib.spec_op_linear_scratch_floats.restype = C.c_size_t
    lib.spec_op_linear_scratch_floats.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_int32]
    lib.spec_set_option.restype = C.c_int
    lib.spec_set_option.argtypes = [C.c_void_p, C.c_int32, C.c_int32]
    lib.spec_trace_read.restype = C.c_int
    lib.spec_trace_read.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.POINTER(C.c_int32)]
    lib.spec_build_labels.restype = C.c_int
    lib.spec_build_labels.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                      C.c_void_p, C.c_void_p]
    lib.spec_op_linear_static.restype = C.c_int
    lib.spec_op_linear_static.argtypes = [C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32,
                                          C.c_int32, C.c_int32, C.c_void_p]
    lib.spec_packed_weight_bytes.restype = C.c_size_t
    lib.spec_packed_weight_bytes.argtypes = [C.c_int32, C.c_int32]
    lib.spec_pack_weight.restype = C.c_int
    lib.spec_pack_weight.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
    lib.spec_last_step_phase_ms.restype = C.c_int
    lib.spec_last_step_phase_ms.argtypes = [C.c_void_p, C.c_void_p]
    lib.spec_debug_wait_timeout.restype = C.c_int
    lib.spec_debug_wait_timeout.argtypes = [C.c_void_p, C.c_int32]
    lib.spec_profile_kernel.restype = C.c_int
    lib.spec_profile_kernel.argtypes = [C.c_void_p, C.c_int32]
    lib.spec_profile_read.restype = C.c_int
    lib.spec_profile_read.argtypes = [C.c_void_p, C.POINTER(C.c_double), C.POINTER(C.c_int64)]
    _lib = lib
    return lib


def _i32ptr(a: np.ndarray):
    return a.ctypes.data_as(C.POINTER(C.c_int32))


def upload_weights(cfg, weights: Dict[str, np.ndarray], device="cuda:0") -> Dict[str, "object"]:
    """float32 numpy tensors -> device tensors of the configuration's operand type (gains stay
    float32). The q, k and v matrices of a layer go into one allocation in that order."""
    import torch
    dt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    out = {}

    def put(a, dtype):
        return torch.from_numpy(np.ascontiguousarray(a)).to(device).to(dtype).contiguous()

    for name in ("embed", "lm_head"):
        out[name] = put(weights[name], dt)
    out["final_norm"] = put(weights["final_norm"], torch.float32)
    for l in range(cfg.n_layers):
        p = f"layers.{l}."
        qkv = np.concatenate([weights[p + "wq"], weights[p + "wk"], weights[p + "wv"]], axis=0)
        out[p + "wqkv"] = put(qkv, dt)
        for nm in ("wo", "w_gate", "w_up", "w_down"):
            out[p + nm] = put(weights[p + nm], dt)
        for nm in ("attn_norm", "ffn_norm"):
            out[p + nm] = put(weights[p + nm], torch.float32)
    for k in range(cfg.n_medusa):
        out[f"medusa.{k}.w"] = put(weights[f"medusa.{k}.w"], dt)
        out[f"medusa.{k}.b"] = put(weights[f"medusa.{k}.b"], dt)
    return out


def spec_pack_weight(w):
    """Pre-tiled image (uint8 CUDA tensor) of a row-major bf16 CUDA matrix, made by the library."""
    import torch
    lib = load_library()
    rows, cols = w.shape
    nbytes = int(lib.spec_packed_weight_bytes(rows, cols))
    if nbytes == 0 or w.dtype != torch.bfloat16 or not w.is_contiguous():
        raise SpecError(-1, "spec_pack_weight: needs a contiguous bf16 matrix whose width is a multiple of 64")
    out = torch.empty(nbytes, dtype=torch.uint8, device=w.device)
    rc = lib.spec_pack_weight(w.data_ptr(), rows, cols, out.data_ptr(), torch.cuda.current_stream(w.device).cuda_stream)
    if rc != 0:
        raise SpecError(rc, lib.spec_last_error(None).decode())
    return out


def pack_linear_weights(cfg, dev_weights: Dict[str, "object"]) -> Dict[str, "object"]:
    """Pre-tiled images of every linear weight of the model (q, k and v separately), keyed like the
    pointers of spec_weights; cached on the weight dictionary, so decoders that share weights share
    the images."""
    cache = dev_weights.get("__packed__")
    if cache is not None:
        return cache
    qrows, krows = cfg.n_heads * cfg.head_dim, cfg.n_kv_heads * cfg.head_dim
    out = {"lm_head": spec_pack_weight(dev_weights["lm_head"])}
    for l in range(cfg.n_layers):
        p = f"layers.{l}."
        qkv = dev_weights[p + "wqkv"]
        out[p + "wq"] = spec_pack_weight(qkv[:qrows])
        out[p + "wk"] = spec_pack_weight(qkv[qrows:qrows + krows])
        out[p + "wv"] = spec_pack_weight(qkv[qrows + krows:])
        for nm in ("wo", "w_gate", "w_up", "w_down"):
            out[p + nm] = spec_pack_weight(dev_weights[p + nm])
    for k in range(cfg.n_medusa):
        out[f"medusa.{k}.w"] = spec_pack_weight(dev_weights[f"medusa.{k}.w"])
    import torch
    torch.cuda.synchronize()      # whatever stream a decoder runs on, the images are complete
    dev_weights["__packed__"] = out
    return out


class SpecDecoder:
    """Owns the device tensors and a spec_ctx; methods mirror the C entry points. On the bf16 tensor-core
    path the linear weights are handed over as pre-tiled images unless packed=False."""

    def __init__(self, cfg, dev_weights: Dict[str, "object"], tree: Dict[str, np.ndarray], max_seq: int,
                 max_batch: int = 1, flags: int = 0, accept_mode: int = 0, typ_eps: float = 0.09,
                 typ_delta: float = 0.3, temperature: float = 1.0, frag_token: int = -1, stream=None,
                 packed: Optional[bool] = None, sampling: bool = False, seed: int = 0):
        import torch
        tc_path = cfg.dtype == "bf16" and not (flags & FLAG_SIMPLE_KERNELS)
        self.packed = tc_path if packed is None else bool(packed)
        if self.packed:
            if not tc_path:
                raise SpecError(-1, "pre-tiled weights need the bf16 tensor-core path")
            flags |= FLAG_PACKED_WEIGHTS
        self.torch = torch
        self.lib = load_library()
        self.cfg = cfg
        self.K = cfg.n_medusa
        self.T = int(len(tree["parent"]))
        self.max_batch = max_batch
        self.w = dev_weights
        self.device = dev_weights["embed"].device
        self._tree = {k: np.ascontiguousarray(tree[k], dtype=np.int32) for k in ("parent", "depth", "rank")}
        self._ctree = SpecTree(self.T, _i32ptr(self._tree["parent"]), _i32ptr(self._tree["depth"]),
                               _i32ptr(self._tree["rank"]))
        self._ccfg = SpecConfig(cfg.n_layers, cfg.d_model, cfg.n_heads, cfg.n_kv_heads, cfg.head_dim, cfg.d_ffn,
                                cfg.vocab, cfg.rms_eps, cfg.rope_base, 1 if cfg.dtype == "bf16" else 0, cfg.n_medusa,
                                max_batch, max_seq, cfg.page_size, accept_mode, typ_eps, typ_delta, temperature,
                                frag_token, flags, 1 if sampling else 0, seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)
        L = cfg.n_layers
        qrows = cfg.n_heads * cfg.head_dim
        krows = cfg.n_kv_heads * cfg.head_dim
        esz = 2 if cfg.dtype == "bf16" else 4

        def arr(ptrs: Sequence[int]):
            a = (C.c_void_p * max(1, len(ptrs)))(*ptrs)
            return a

        lw = lambda nm: [dev_weights[f"layers.{l}.{nm}"].data_ptr() for l in range(L)]
        if self.packed:
            self._pk = pack_linear_weights(cfg, dev_weights)
            pw = lambda nm: [self._pk[f"layers.{l}.{nm}"].data_ptr() for l in range(L)]
            lin = {nm: pw(nm) for nm in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down")}
            medusa_w = [self._pk[f"medusa.{k}.w"].data_ptr() for k in range(self.K)]
            lm_head_ptr = self._pk["lm_head"].data_ptr()
        else:
            qkv = lw("wqkv")
            lin = {"wq": qkv, "wk": [p + qrows * cfg.d_model * esz for p in qkv],
                   "wv": [p + (qrows + krows) * cfg.d_model * esz for p in qkv],
                   "wo": lw("wo"), "w_gate": lw("w_gate"), "w_up": lw("w_up"), "w_down": lw("w_down")}
            medusa_w = [dev_weights[f"medusa.{k}.w"].data_ptr() for k in range(self.K)]
            lm_head_ptr = dev_weights["lm_head"].data_ptr()
        self._arrs = {
            "attn_norm": arr(lw("attn_norm")), "wq": arr(lin["wq"]), "wk": arr(lin["wk"]), "wv": arr(lin["wv"]),
            "wo": arr(lin["wo"]), "ffn_norm": arr(lw("ffn_norm")), "w_gate": arr(lin["w_gate"]),
            "w_up": arr(lin["w_up"]), "w_down": arr(lin["w_down"]),
            "medusa_w": arr(medusa_w),
            "medusa_b": arr([dev_weights[f"medusa.{k}.b"].data_ptr() for k in range(self.K)]),
        }
        self._cw = SpecWeights(dev_weights["embed"].data_ptr(), lm_head_ptr,
                               dev_weights["final_norm"].data_ptr(),
                               *[C.cast(self._arrs[n], C.POINTER(C.c_void_p)) for n in
                                 ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down",
                                  "medusa_w", "medusa_b")])
        nbytes = self.lib.spec_workspace_bytes(C.byref(self._ccfg), C.byref(self._ctree))
        if nbytes == 0:
            raise SpecError(-1, "spec_workspace_bytes rejected the configuration or tree")
        self.workspace_bytes = int(nbytes)
        self.workspace = torch.empty(self.workspace_bytes + 1024, dtype=torch.uint8, device=self.device)
        base = (self.workspace.data_ptr() + 1023) // 1024 * 1024
        self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        self._ctx = C.c_void_p()
        rc = self.lib.spec_create(C.byref(self._ccfg), C.byref(self._cw), C.byref(self._ctree), base,
                                  self.workspace_bytes, self.stream.cuda_stream, C.byref(self._ctx))
        if rc != 0:
            raise SpecError(rc, self.lib.spec_last_error(None).decode())
        self.kmax = int(self.lib.spec_query(self._ctx, Q_KMAX))
        self.batch = max_batch
        self._out_tok = torch.empty((max_batch, self.K + 1), dtype=torch.int32).pin_memory()
        self._out_cnt = torch.empty((max_batch,), dtype=torch.int32).pin_memory()
        self._ov = torch.empty((max_batch, max(self.K, 1), self.kmax), dtype=torch.int32).pin_memory()

    def _check(self, rc: int):
        if rc != 0:
            raise SpecError(rc, self.lib.spec_last_error(self._ctx).decode())

    def close(self):
        if self._ctx:
            self.lib.spec_destroy(self._ctx)
            self._ctx = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def prefill(self, prompts):
        """prompts: one int array or a list of them (one per sequence)."""
        if isinstance(prompts, np.ndarray) and prompts.ndim == 1:
            prompts = [prompts]
        toks = np.ascontiguousarray(np.concatenate([np.asarray(p, dtype=np.int32) for p in prompts]))
        offs = np.zeros(len(prompts) + 1, dtype=np.int32)
        offs[1:] = np.cumsum([len(p) for p in prompts])
        self.batch = len(prompts)
        self._check(self.lib.spec_prefill(self._ctx, self.batch, toks.ctypes.data, offs.ctypes.data))

    def step(self, cand_override: Optional[np.ndarray] = None):
        """One synchronous step; returns (tokens [batch][K+1] int32, counts [batch])."""
        ov = None
        if cand_override is not None:
            self._ov[: self.batch].copy_(self.torch.from_numpy(
                np.ascontiguousarray(cand_override, dtype=np.int32).reshape(self.batch, self.K, self.kmax)))
            ov = self._ov.data_ptr()
        self._check(self.lib.spec_step(self._ctx, self._out_tok.data_ptr(), self._out_cnt.data_ptr(), ov))
        return self._out_tok[: self.batch].numpy().copy(), self._out_cnt[: self.batch].numpy().copy()

    def step_async(self):
        """Enqueue one step on the stream without host synchronisation."""
        self._check(self.lib.spec_step(self._ctx, None, None, None))

    def read_generated(self, seq: int = 0, max_tokens: int = 1 << 16) -> np.ndarray:
        buf = np.zeros(max_tokens, dtype=np.int32)
        n = C.c_int32(0)
        self._check(self.lib.spec_read_generated(self._ctx, seq, buf.ctypes.data, max_tokens, C.byref(n)))
        return buf[: min(n.value, max_tokens)].copy()

    def phase_ms(self) -> np.ndarray:
        """Device milliseconds of the last step's five parts (heads, expand, verify, accept, compact)."""
        ms = np.zeros(5, dtype=np.float32)
        self._check(self.lib.spec_last_step_phase_ms(self._ctx, ms.ctypes.data))
        return ms

    def profile_kernel(self, kind: int):
        self._check(self.lib.spec_profile_kernel(self._ctx, kind))

    def profile_read(self):
        ms, n = C.c_double(0.0), C.c_int64(0)
        self._check(self.lib.spec_profile_read(self._ctx, C.byref(ms), C.byref(n)))
        return ms.value, n.value

    def trace(self, max_records: int = 1024):
        """Timeline of the last step (OPT_TRACE must be on): list of (name, start, end, mark_a, mark_b) in ns."""
        names = C.create_string_buffer(max_records * TRACE_NAME_LEN)
        stamps = np.zeros((max_records, 4), dtype=np.uint64)
        n = C.c_int32(0)
        self._check(self.lib.spec_trace_read(self._ctx, max_records, names, stamps.ctypes.data, C.byref(n)))
        out = []
        for i in range(min(n.value, max_records)):
            nm = names.raw[i * TRACE_NAME_LEN:(i + 1) * TRACE_NAME_LEN].split(b"\0")[0].decode()
            out.append((nm,) + tuple(int(v) for v in stamps[i]))
        return out

    def wait_timeout_probe(self, limit_us: int) -> int:
        """Runs the bounded-wait self test; returns the library's code (SPEC_E_TIMEOUT = -6 when it works)."""
        return int(self.lib.spec_debug_wait_timeout(self._ctx, limit_us))

    def set_option(self, what: int, value: int):
        self._check(self.lib.spec_set_option(self._ctx, what, value))

    def gate_up_kernel_name(self) -> str:
        """Name of the kernel a step's gate+up projection runs as (the dominant kernel of a 7B step)."""
        m = self.batch * self.T
        mt = 16 if m <= 16 else (32 if m <= 32 else (64 if m <= 64 else 128))
        if self.query(Q_CLUSTER_GATE_UP):
            return f"gemm_cluster<{mt},swiglu>"
        return "gemm_wide" if m > 128 and self.query(Q_WIDE_GEMM) else f"gemm_stream<{mt}>"

    def query(self, what: int) -> int:
        return int(self.lib.spec_query(self._ctx, what))

    def debug(self, what: int) -> np.ndarray:
        rows = self.batch * self.T
        shapes = {DBG_TOK: ((rows,), np.int32), DBG_POS: ((rows,), np.int32),
                  DBG_LOGITS: ((rows, self.cfg.vocab), np.float32), DBG_HIDDEN: ((rows, self.cfg.d_model), np.float32),
                  DBG_ARGMAX: ((rows,), np.int32), DBG_PATH: ((self.batch, self.K + 1), np.int32),
                  DBG_CAND: ((self.batch, self.K + 1, self.kmax), np.int32), DBG_SEQLEN: ((self.batch,), np.int32),
                  DBG_NEXT_ROOT: ((self.batch,), np.int32), DBG_H_LAST: ((self.batch, self.cfg.d_model), np.float32),
                  DBG_STATUS: ((4,), np.int32)}
        shape, dt = shapes[what]
        buf = np.zeros(shape, dtype=dt)
        self._check(self.lib.spec_debug_read(self._ctx, what, buf.ctypes.data, buf.nbytes))
        return buf

    def read_kv(self, seq: int, layer: int, slot0: int, n_slots: int):
        shape = (n_slots, self.cfg.n_kv_heads, self.cfg.head_dim)
        k, v = np.zeros(shape, np.float32), np.zeros(shape, np.float32)
        self._check(self.lib.spec_debug_read_kv(self._ctx, seq, layer, slot0, n_slots, k.ctypes.data, v.ctypes.data))
        return k, v


def spec_op_linear(x, w, ctas: int = 296):
    """y = x @ w.T through the library's linear kernel (x, w: CUDA tensors, float32 or bf16)."""
    import torch
    lib = load_library()
    M, K = x.shape
    N = w.shape[0]
    dtype = 1 if x.dtype == torch.bfloat16 else 0
    y = torch.empty((M, N), dtype=torch.float32, device=x.device)
    scratch = None
    if dtype == 1:
        need = int(lib.spec_op_linear_scratch_floats(M, N, K, ctas))
        if need == 0:
            raise SpecError(-1, "spec_op_linear_scratch_floats rejected the shape")
        scratch = torch.empty(need + 4, dtype=torch.float32, device=x.device)
    rc = lib.spec_op_linear(dtype, x.data_ptr(), w.data_ptr(), y.data_ptr(), M, N, K, ctas,
                            scratch.data_ptr() if scratch is not None else None,
                            torch.cuda.current_stream(x.device).cuda_stream)
    if rc != 0:
        raise SpecError(rc, "spec_op_linear failed")
    return y


def spec_build_labels(tokens, num_heads: int, frag: int, pad: int, ignore: int):
    """tokens: CUDA int32 tensor [n_seq, seq_len] -> labels [n_seq, num_heads + 1, seq_len] (Sec. III-C)."""
    import torch
    lib = load_library()
    n_seq, seq_len = tokens.shape
    labels = torch.empty((n_seq, num_heads + 1, seq_len), dtype=torch.int32, device=tokens.device)
    rc = lib.spec_build_labels(tokens.data_ptr(), n_seq, seq_len, num_heads, frag, pad, ignore, labels.data_ptr(),
                               torch.cuda.current_stream(tokens.device).cuda_stream)
    if rc != 0:
        raise SpecError(rc, "spec_build_labels failed")
    return labels


STATIC_SCRATCH_FLOATS = 2 << 20


def spec_op_linear_static(x, w, y, ctas: int = 296):
    """y[M,N] (float32, preallocated by the caller) = x @ w.T through the entry point that keeps
    its scratch inside the library. For callers that may not allocate device memory: nothing
    is allocated here either, the three tensors are used as given. Raises SpecError with the
    library's message when the shape needs more than STATIC_SCRATCH_FLOATS of partial sums."""
    import torch
    lib = load_library()
    M, K = x.shape
    N = w.shape[0]
    dtype = 1 if x.dtype == torch.bfloat16 else 0
    rc = lib.spec_op_linear_static(dtype, x.data_ptr(), w.data_ptr(), y.data_ptr(), M, N, K, ctas,
                                   torch.cuda.current_stream(x.device).cuda_stream)
    if rc != 0:
        raise SpecError(rc, lib.spec_last_error(None).decode())
    return y
