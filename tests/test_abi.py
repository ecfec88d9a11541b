"""The C-ABI library loads, exports every declared symbol and validates its arguments (no GPU)."""
import ctypes as C
import os
import re

import pytest

import inputs
from paper_2406_13170_b200 import binding as b
from paper_2406_13170_b200 import build as amph_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    amph_build.build()
    return b.lib()


def test_exports_every_declared_symbol(L):
    header = open(os.path.join(ROOT, "include", "amph.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(amph_[a-z_]+)\s*\(", header))
    assert {"amph_init", "amph_load_weights", "amph_prefill", "amph_draft", "amph_verify_tree",
            "amph_accept", "amph_step"} <= declared
    for name in declared:
        assert hasattr(L, name), f"{name} is declared in amph.h but not exported"
    assert declared == set(b.EXPORTS)


def _cfg_tree(shape_name="tiny"):
    s = inputs.get_shape(shape_name)
    topo = inputs.make_tree(s.n_nodes, s.topk)
    return s, b.make_config(s), b.make_tree(topo)


def test_workspace_bytes_and_shape_errors(L):
    s, cfg, tr = _cfg_tree("7b")
    kv, ws = C.c_size_t(), C.c_size_t()
    assert L.amph_workspace_bytes(C.byref(cfg), C.byref(tr.c), C.byref(kv), C.byref(ws)) == 0
    per_layer = 2 * s.n_heads * cfg.max_ctx * s.head_dim * 2
    assert kv.value == per_layer * (s.n_layers + s.n_sal)
    assert ws.value > 0 and ws.value % 256 == 0
    cfg.head_dim = 96
    assert L.amph_workspace_bytes(C.byref(cfg), C.byref(tr.c), C.byref(kv), C.byref(ws)) == 2
    assert b"head_dim" in L.amph_last_error(None)
    s, cfg, tr = _cfg_tree()
    cfg.kv_dtype = 1 - cfg.weight_dtype
    assert L.amph_workspace_bytes(C.byref(cfg), C.byref(tr.c), C.byref(kv), C.byref(ws)) == 2
    s, cfg, tr = _cfg_tree()
    cfg.topk[0] = 1                       # the tree uses rank 3 at depth 1
    assert L.amph_workspace_bytes(C.byref(cfg), C.byref(tr.c), C.byref(kv), C.byref(ws)) == 2
    assert b"rank" in L.amph_last_error(None)
    s, cfg, tr = _cfg_tree()
    tr.parent[3] = 5                      # parent after child
    assert L.amph_workspace_bytes(C.byref(cfg), C.byref(tr.c), C.byref(kv), C.byref(ws)) == 2
    assert L.amph_workspace_bytes(None, C.byref(tr.c), C.byref(kv), C.byref(ws)) == 1


def test_null_context_calls_fail_cleanly(L):
    assert L.amph_step(None, None, None) == 1
    assert L.amph_draft(None, None, None) == 1
    assert L.amph_get_state(None, None, None, None) == 1
    L.amph_destroy(None)
    out = C.c_void_p()
    s, cfg, tr = _cfg_tree()
    assert L.amph_init(C.byref(cfg), C.byref(tr.c), None, 0, None, 0, None, C.byref(out)) == 1
    assert not out.value
    # misaligned / undersized regions are rejected before any device call
    assert L.amph_init(C.byref(cfg), C.byref(tr.c), C.c_void_p(0x1001), 1 << 40, C.c_void_p(0x2000), 1 << 40,
                       None, C.byref(out)) == 5
    assert L.amph_init(C.byref(cfg), C.byref(tr.c), C.c_void_p(0x1000), 16, C.c_void_p(0x2000), 16,
                       None, C.byref(out)) == 5


def test_no_device_means_error_not_fallback(L):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    out = C.c_void_p()
    s, cfg, tr = _cfg_tree()
    rc = L.amph_init(C.byref(cfg), C.byref(tr.c), C.c_void_p(0x1000), 1 << 40, C.c_void_p(0x100000), 1 << 40,
                     None, C.byref(out))
    assert rc == 7 and b"no CUDA device" in L.amph_last_error(None)
