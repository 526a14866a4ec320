"""The C-ABI library loads and exports every function the header declares (no GPU needed),
and its host-side validation rejects bad configurations and trees."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2503_14153_b200 import binding as B
from paper_2503_14153_b200 import build_tree
from synthetic import get_config

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2503_14153_b200 import build
    build.build()
    return B.load_library()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "spec_decode.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(spec_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_functions()
    assert set(names) == set(B.EXPORTS)
    for n in names:
        assert hasattr(lib, n), n


def _cfg_struct(cfg, **kw):
    vals = dict(n_layers=cfg.n_layers, d_model=cfg.d_model, n_heads=cfg.n_heads, n_kv_heads=cfg.n_kv_heads,
                head_dim=cfg.head_dim, d_ffn=cfg.d_ffn, vocab=cfg.vocab, rms_eps=cfg.rms_eps, rope_base=cfg.rope_base,
                dtype=1 if cfg.dtype == "bf16" else 0, n_medusa=cfg.n_medusa, max_batch=1, max_seq=128,
                page_size=16, accept_mode=0, typ_eps=0.09, typ_delta=0.3, temperature=1.0, frag_token=-1, flags=0)
    vals.update(kw)
    return B.SpecConfig(**vals)


def _tree_struct(tree):
    arrs = [np.ascontiguousarray(tree[k], dtype=np.int32) for k in ("parent", "depth", "rank")]
    t = B.SpecTree(len(arrs[0]), *[a.ctypes.data_as(C.POINTER(C.c_int32)) for a in arrs])
    t._keep = arrs
    return t


def test_workspace_bytes_grows_with_shape_and_rejects_bad_input(lib):
    c0 = get_config("c0")
    tree = _tree_struct(build_tree(c0.topk, c0.tree_nodes))
    a = lib.spec_workspace_bytes(C.byref(_cfg_struct(c0)), C.byref(tree))
    b = lib.spec_workspace_bytes(C.byref(_cfg_struct(c0, max_seq=1024)), C.byref(tree))
    assert 0 < a < b
    c1 = get_config("c1")
    t1 = _tree_struct(build_tree(c1.topk, c1.tree_nodes))
    big = lib.spec_workspace_bytes(C.byref(_cfg_struct(c1, max_seq=8192 + 256)), C.byref(t1))
    kv = (8192 + 256) * 32 * 2 * 32 * 128 * 2
    assert kv < big < kv + 4 * 2 ** 30
    assert lib.spec_workspace_bytes(C.byref(_cfg_struct(c0, dtype=3)), C.byref(tree)) == 0
    assert lib.spec_workspace_bytes(C.byref(_cfg_struct(c0, n_heads=3, n_kv_heads=2)), C.byref(tree)) == 0
    assert lib.spec_workspace_bytes(C.byref(_cfg_struct(c1, page_size=8)), C.byref(t1)) == 0
    assert lib.spec_workspace_bytes(None, C.byref(tree)) == 0


@pytest.mark.parametrize("mutate", [
    lambda p, d, r: p.__setitem__(0, 0),          # root must have parent -1
    lambda p, d, r: p.__setitem__(2, 5),          # parent after child
    lambda p, d, r: d.__setitem__(3, 9),          # depth not parent's + 1
    lambda p, d, r: r.__setitem__(1, 99),         # rank out of range
    lambda p, d, r: r.__setitem__(2, int(r[1])),  # siblings share a rank
])
def test_bad_trees_are_rejected(lib, mutate):
    c0 = get_config("c0")
    tree = build_tree(c0.topk, c0.tree_nodes)
    p, d, r = tree["parent"].copy(), tree["depth"].copy(), tree["rank"].copy()
    mutate(p, d, r)
    assert lib.spec_workspace_bytes(C.byref(_cfg_struct(c0)), C.byref(_tree_struct({"parent": p, "depth": d, "rank": r}))) == 0


def test_tree_deeper_than_heads_is_rejected(lib):
    c0 = get_config("c0")
    assert lib.spec_workspace_bytes(C.byref(_cfg_struct(c0, n_medusa=2)),
                                    C.byref(_tree_struct(build_tree(c0.topk, c0.tree_nodes)))) == 0


def test_null_context_calls_fail_cleanly(lib):
    assert lib.spec_step(None, None, None, None) == -1
    assert lib.spec_prefill(None, 1, None, None) == -1
    assert lib.spec_destroy(None) == -1
    assert lib.spec_query(None, 0) == -1
    assert lib.spec_last_error(None) is not None


def test_product_tree_matches_oracle_tree():
    from oracle.tree import build_tree as oracle_tree
    for caps, T in [((4, 2, 2), 16), ((10, 4, 2, 2), 16), ((10, 4, 2, 2), 32), ((10, 4, 2, 2), 64),
                    ((10, 4, 2, 2), 128), ((3, 3), 12), ((2,), 3), ((5, 5, 5), 1)]:
        a, b = build_tree(caps, T), oracle_tree(caps, T)
        for k in ("parent", "depth", "rank"):
            assert np.array_equal(a[k], b[k]), (caps, T, k)
