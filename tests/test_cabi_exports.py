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


def test_newer_entry_points_validate_on_the_host_too():
    import paper_2512_22737_b200 as w
    lib = w.load_library()
    ok = w.make_config(batch=2, window=32, n_q_heads=32, n_kv_heads=8, head_dim=128, page_size=16, max_pages_per_seq=8,
                       num_pages=32, max_prefix_len=64, vocab=4096, mask_token_id=4095)
    # whole step from host buffers: sizes, then null pointers
    assert w.wedlm_step_host_workspace_bytes(ok) > w.wedlm_window_attn_workspace_bytes(ok) + w.wedlm_confidence_workspace_bytes(ok)
    nulls = [None] * 15
    assert lib.wedlm_step_host(ctypes.byref(ok), *nulls, None, 0, None, None, None) == -1
    # Dual-Stream Masking: blocks must own whole pages; n_blocks must match the sequence length
    assert w.wedlm_dual_stream_workspace_bytes(ok, 4) > 0
    odd = w.make_config(batch=2, window=24, n_q_heads=32, n_kv_heads=8, head_dim=128, page_size=16, vocab=4096)
    assert w.wedlm_dual_stream_workspace_bytes(odd, 4) == 0
    assert lib.wedlm_dual_stream_attn(ctypes.byref(odd), 4, None, None, None, None, None, None, 0, None, None) == -2
    assert lib.wedlm_dual_stream_construct(ctypes.byref(ok), 4, 200, None, None, None, None, None, None, None) == -1   # 200 > 4 * 32
    assert lib.wedlm_dual_stream_construct(ctypes.byref(ok), 4, 96, None, None, None, None, None, None, None) == -1    # 96 fits 3 blocks
    assert lib.wedlm_dual_stream_construct(ctypes.byref(ok), 4, 100, None, None, None, None, None, None, None) == -1   # null pointers
    # sampling: a negative or non-finite temperature is refused, a positive one enlarges the workspace
    hot = w.make_config(batch=2, window=32, vocab=4096, sample_temperature=0.5)
    cold = w.make_config(batch=2, window=32, vocab=4096)
    assert w.wedlm_confidence_workspace_bytes(hot) > w.wedlm_confidence_workspace_bytes(cold) > 0
    for bad in (-0.1, float("nan"), float("inf")):
        assert w.wedlm_confidence_workspace_bytes(w.make_config(batch=2, window=32, vocab=4096, sample_temperature=bad)) == 0
