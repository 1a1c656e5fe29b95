"""The C-ABI library loads on a machine without a GPU and exports every symbol the header declares.
No compute call is made here."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "wedlm.h")


def _declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(wedlm_[a-z_]+)\s*\(", text)))


@pytest.fixture(scope="module")
def lib():
    from paper_2512_22737_b200 import build
    path = build.build()
    return ctypes.CDLL(path)


def test_header_declares_the_entry_points_of_the_step():
    names = _declared_functions()
    for want in ["wedlm_reorder", "wedlm_window_attn", "wedlm_kv_append", "wedlm_confidence_commit",
                 "wedlm_window_refill", "wedlm_window_attn_workspace_bytes",
                 "wedlm_confidence_workspace_bytes", "wedlm_strerror", "wedlm_version"]:
        assert want in names


def test_every_declared_symbol_is_exported(lib):
    for name in _declared_functions():
        assert hasattr(lib, name), name


def test_strerror_and_version_run_without_a_gpu(lib):
    lib.wedlm_strerror.restype = ctypes.c_char_p
    assert lib.wedlm_strerror(0) == b"ok"
    assert b"invalid" in lib.wedlm_strerror(-1)
    assert lib.wedlm_version() >= 100


def test_argument_validation_happens_on_the_host():
    """Bad configs are rejected before any launch, so this needs no device."""
    import paper_2512_22737_b200 as w
    w.load_library()
    lib = w.load_library()
    cfg = w.make_config(batch=1, window=0)
    assert lib.wedlm_reorder(ctypes.byref(cfg), None, None, None, None, None, None, None, None, None, None, None) == -1
    cfg = w.make_config(batch=1, window=8, n_q_heads=3, n_kv_heads=2, head_dim=64, max_pages_per_seq=4, num_pages=4)
    assert w.wedlm_window_attn_workspace_bytes(cfg) == 0          # heads do not divide
    cfg = w.make_config(batch=1, window=8, n_q_heads=4, n_kv_heads=2, head_dim=48, max_pages_per_seq=4, num_pages=4)
    assert w.wedlm_window_attn_workspace_bytes(cfg) == 0          # unsupported head size
    cfg = w.make_config(batch=1, window=8, n_q_heads=4, n_kv_heads=2, head_dim=64, max_pages_per_seq=4,
                        num_pages=4, max_prefix_len=60)
    assert w.wedlm_window_attn_workspace_bytes(cfg) == 0          # prefix + window exceeds the block table
    cfg = w.make_config(batch=1, window=8, n_q_heads=4, n_kv_heads=2, head_dim=64, max_pages_per_seq=5,
                        num_pages=8, max_prefix_len=64, vocab=1001, dtype="f32")
    assert w.wedlm_window_attn_workspace_bytes(cfg) > 0
    assert w.wedlm_confidence_workspace_bytes(cfg) > 0
    # null pointers
    assert lib.wedlm_reorder(ctypes.byref(cfg), None, None, None, None, None, None, None, None, None, None, None) == -1
    # empty batch is a no-op
    cfg0 = w.make_config(batch=0, window=8)
    assert lib.wedlm_reorder(ctypes.byref(cfg0), None, None, None, None, None, None, None, None, None, None, None) == 0
