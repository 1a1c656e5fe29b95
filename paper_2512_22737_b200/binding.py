"""ctypes binding over libwedlm.so: argument marshalling only.

Every function mirrors the C entry point of the same name in ``include/wedlm.h``.  Tensors are
torch CUDA tensors (they provide device memory and the stream); this module checks dtype /
device / contiguity, extracts raw pointers and calls the library.  All arithmetic of the step
runs inside the library's kernels.
"""
from __future__ import annotations

import ctypes
import math
import os
from typing import Dict, Optional

import numpy as np
import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "lib", "libwedlm.so")
_lib = None

WEDLM_DTYPE_BF16, WEDLM_DTYPE_F32 = 0, 1
WEDLM_CONF_ENTROPY, WEDLM_CONF_MAXPROB = 0, 1
WEDLM_ATTN_AUTO, WEDLM_ATTN_GENERIC, WEDLM_ATTN_TENSOR = 0, 1, 2
WEDLM_STATUS_BAD_PAGE, WEDLM_STATUS_BAD_LENGTH, WEDLM_STATUS_WAIT_EXPIRED = 1, 2, 4


class WedlmError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {wedlm_strerror(code)} ({code})")


class WedlmConfig(ctypes.Structure):
    """Mirror of wedlm_config_t."""
    _fields_ = [
        ("batch", ctypes.c_int32), ("window", ctypes.c_int32), ("n_q_heads", ctypes.c_int32),
        ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("page_size", ctypes.c_int32),
        ("max_pages_per_seq", ctypes.c_int32), ("num_pages", ctypes.c_int32), ("vocab", ctypes.c_int32),
        ("dtype", ctypes.c_int32), ("rope_style", ctypes.c_int32), ("rope_theta", ctypes.c_float),
        ("softmax_scale", ctypes.c_float), ("conf_mode", ctypes.c_int32), ("tau", ctypes.c_float),
        ("lambda_", ctypes.c_float), ("maxprob_thr", ctypes.c_float), ("mask_token_id", ctypes.c_int32),
        ("max_prefix_len", ctypes.c_int32), ("attn_impl", ctypes.c_int32), ("commit_mode", ctypes.c_int32),
        ("sample_temperature", ctypes.c_float), ("sample_seed_lo", ctypes.c_uint32), ("sample_seed_hi", ctypes.c_uint32),
    ]

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.bfloat16 if self.dtype == WEDLM_DTYPE_BF16 else torch.float32


def library_path() -> str:
    return _LIB_PATH


def load_library() -> ctypes.CDLL:
    """Load libwedlm.so.  Raises if it has not been built: there is no fallback path."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(
            f"{_LIB_PATH} is missing: build it with `python -m paper_2512_22737_b200.build` "
            "(needs nvcc).  This package has no CPU or PyTorch fallback.")
    lib = ctypes.CDLL(_LIB_PATH)
    vp, i32p, u8p, f32p = ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p
    cfgp = ctypes.POINTER(WedlmConfig)
    lib.wedlm_strerror.restype = ctypes.c_char_p
    lib.wedlm_strerror.argtypes = [ctypes.c_int]
    lib.wedlm_version.restype = ctypes.c_int
    lib.wedlm_version.argtypes = []
    lib.wedlm_launch_count.restype = ctypes.c_ulonglong
    lib.wedlm_launch_count.argtypes = []
    lib.wedlm_profile_next_attn.restype = ctypes.c_int
    lib.wedlm_profile_next_attn.argtypes = [vp, vp]
    lib.wedlm_selftest_wait_expiry.restype = ctypes.c_int
    lib.wedlm_selftest_wait_expiry.argtypes = [ctypes.c_uint32, i32p, vp]
    lib.wedlm_reorder.restype = ctypes.c_int
    lib.wedlm_reorder.argtypes = [cfgp, u8p, i32p, i32p, i32p, i32p, i32p, i32p, i32p, i32p, i32p, vp]
    lib.wedlm_window_attn_workspace_bytes.restype = ctypes.c_size_t
    lib.wedlm_window_attn_workspace_bytes.argtypes = [cfgp]
    lib.wedlm_window_attn.restype = ctypes.c_int
    lib.wedlm_window_attn.argtypes = [cfgp, vp, vp, vp, vp, vp, i32p, i32p, i32p, vp, i32p, vp,
                                      ctypes.c_size_t, i32p, vp]
    lib.wedlm_kv_append.restype = ctypes.c_int
    lib.wedlm_kv_append.argtypes = [cfgp, vp, vp, i32p, vp, vp, i32p, i32p, i32p, i32p, i32p, vp]
    lib.wedlm_confidence_workspace_bytes.restype = ctypes.c_size_t
    lib.wedlm_confidence_workspace_bytes.argtypes = [cfgp]
    lib.wedlm_confidence_commit.restype = ctypes.c_int
    lib.wedlm_confidence_commit.argtypes = [cfgp, vp, i32p, i32p, i32p, i32p, u8p, i32p, i32p, i32p,
                                            i32p, f32p, f32p, f32p, i32p, i32p, i32p, vp,
                                            ctypes.c_size_t, i32p, vp]
    lib.wedlm_confidence_commit_static.restype = ctypes.c_int
    lib.wedlm_confidence_commit_static.argtypes = [cfgp, vp, i32p, i32p, i32p, i32p, u8p, i32p, i32p, i32p,
                                                   i32p, f32p, f32p, f32p, i32p, i32p, i32p, i32p, vp]
    lib.wedlm_lmhead_confidence_workspace_bytes.restype = ctypes.c_size_t
    lib.wedlm_lmhead_confidence_workspace_bytes.argtypes = [cfgp, ctypes.c_int32]
    lib.wedlm_lmhead_confidence_commit.restype = ctypes.c_int
    lib.wedlm_lmhead_confidence_commit.argtypes = [cfgp, ctypes.c_int32, vp, vp, i32p, ctypes.c_float, i32p, i32p, i32p,
                                                   i32p, u8p, i32p, i32p, i32p, i32p, f32p, f32p, f32p, i32p, i32p,
                                                   i32p, vp, ctypes.c_size_t, i32p, vp]
    lib.wedlm_window_refill.restype = ctypes.c_int
    lib.wedlm_window_refill.argtypes = [cfgp, i32p, i32p, u8p, i32p, i32p, i32p, i32p, i32p, vp]
    lib.wedlm_step_host_workspace_bytes.restype = ctypes.c_size_t
    lib.wedlm_step_host_workspace_bytes.argtypes = [cfgp]
    lib.wedlm_step_host.restype = ctypes.c_int
    lib.wedlm_step_host.argtypes = [cfgp] + [vp] * 15 + [vp, ctypes.c_size_t, ctypes.POINTER(ctypes.c_void_p), i32p, vp]
    lib.wedlm_step_host_lmhead_workspace_bytes.restype = ctypes.c_size_t
    lib.wedlm_step_host_lmhead_workspace_bytes.argtypes = [cfgp, ctypes.c_int32]
    lib.wedlm_step_host_lmhead.restype = ctypes.c_int
    lib.wedlm_step_host_lmhead.argtypes = [cfgp, ctypes.c_int32] + [vp] * 12 + [ctypes.c_float] + [vp] * 5 + \
                                          [vp, ctypes.c_size_t, ctypes.POINTER(ctypes.c_void_p), i32p, vp]
    lib.wedlm_dual_stream_construct.restype = ctypes.c_int
    lib.wedlm_dual_stream_construct.argtypes = [cfgp, ctypes.c_int32, ctypes.c_int32, i32p, u8p, i32p, i32p, u8p, i32p, vp]
    lib.wedlm_dual_stream_workspace_bytes.restype = ctypes.c_size_t
    lib.wedlm_dual_stream_workspace_bytes.argtypes = [cfgp, ctypes.c_int32]
    lib.wedlm_dual_stream_attn.restype = ctypes.c_int
    lib.wedlm_dual_stream_attn.argtypes = [cfgp, ctypes.c_int32, vp, vp, vp, i32p, vp, vp, ctypes.c_size_t, i32p, vp]
    _lib = lib
    return lib


def wedlm_strerror(code: int) -> str:
    return load_library().wedlm_strerror(int(code)).decode()


def wedlm_version() -> int:
    return int(load_library().wedlm_version())


def wedlm_launch_count() -> int:
    return int(load_library().wedlm_launch_count())


def wedlm_profile_next_attn(event_before: Optional[torch.cuda.Event], event_after: Optional[torch.cuda.Event]) -> None:
    """The events must have been created with enable_timing=True; they are recorded by the next
    wedlm_window_attn call of this thread around its main kernel."""
    def handle(ev):
        if ev is None:
            return None
        if not ev.cuda_event:          # torch creates the handle lazily, on first record
            ev.record()
        return ctypes.c_void_p(ev.cuda_event)
    _check(load_library().wedlm_profile_next_attn(handle(event_before), handle(event_after)),
           "wedlm_profile_next_attn")


def wedlm_selftest_wait_expiry(max_polls: int, status: torch.Tensor, stream=None) -> None:
    _check(load_library().wedlm_selftest_wait_expiry(ctypes.c_uint32(max_polls), _ptr(status, torch.int32, "status"),
                                                     _stream(stream)), "wedlm_selftest_wait_expiry")


def make_config(*, batch, window, n_q_heads=1, n_kv_heads=1, head_dim=128, page_size=16,
                max_pages_per_seq=1, num_pages=1, vocab=1, dtype="bf16", rope_style=0,
                rope_theta=1.0e6, softmax_scale=0.0, conf_mode="entropy", tau=0.3, lam=0.1,
                maxprob_thr=0.9, mask_token_id=0, max_prefix_len=0, attn_impl="auto",
                commit_mode="streaming", sample_temperature=0.0, sample_seed=0) -> WedlmConfig:
    c = WedlmConfig()
    c.batch, c.window, c.n_q_heads, c.n_kv_heads, c.head_dim = batch, window, n_q_heads, n_kv_heads, head_dim
    c.page_size, c.max_pages_per_seq, c.num_pages, c.vocab = page_size, max_pages_per_seq, num_pages, vocab
    c.dtype = {"bf16": WEDLM_DTYPE_BF16, "f32": WEDLM_DTYPE_F32}[dtype]
    c.rope_style, c.rope_theta, c.softmax_scale = rope_style, rope_theta, softmax_scale
    c.conf_mode = {"entropy": WEDLM_CONF_ENTROPY, "maxprob": WEDLM_CONF_MAXPROB}[conf_mode]
    c.tau, c.lambda_, c.maxprob_thr, c.mask_token_id = tau, lam, maxprob_thr, mask_token_id
    c.max_prefix_len = max_prefix_len
    c.attn_impl = {"auto": WEDLM_ATTN_AUTO, "generic": WEDLM_ATTN_GENERIC, "tensor": WEDLM_ATTN_TENSOR}[attn_impl]
    c.commit_mode = {"streaming": 0, "block": 1}[commit_mode]
    c.sample_temperature = sample_temperature
    c.sample_seed_lo, c.sample_seed_hi = sample_seed & 0xFFFFFFFF, (sample_seed >> 32) & 0xFFFFFFFF
    return c


# ----------------------------------------------------------------------------------------
# marshalling helpers
# ----------------------------------------------------------------------------------------
def _ptr(t: Optional[torch.Tensor], dtype: Optional[torch.dtype], name: str):
    if t is None:
        return None
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name} must have dtype {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _check(rc: int, where: str) -> None:
    if rc != 0:
        raise WedlmError(rc, where)


def wedlm_reorder(cfg, filled, window_tokens, prefix_len, window_len, perm, inv_perm, pos_ids,
                  tokens_phys, n_filled, n_commit, stream=None) -> None:
    i32, u8 = torch.int32, torch.uint8
    _check(load_library().wedlm_reorder(
        ctypes.byref(cfg), _ptr(filled, u8, "filled"), _ptr(window_tokens, i32, "window_tokens"),
        _ptr(prefix_len, i32, "prefix_len"), _ptr(window_len, i32, "window_len"), _ptr(perm, i32, "perm"),
        _ptr(inv_perm, i32, "inv_perm"), _ptr(pos_ids, i32, "pos_ids"), _ptr(tokens_phys, i32, "tokens_phys"),
        _ptr(n_filled, i32, "n_filled"), _ptr(n_commit, i32, "n_commit"), _stream(stream)), "wedlm_reorder")


def wedlm_window_attn_workspace_bytes(cfg) -> int:
    return int(load_library().wedlm_window_attn_workspace_bytes(ctypes.byref(cfg)))


def wedlm_window_attn(cfg, q, k, v, k_cache, v_cache, block_table, prefix_len, pos_ids, out,
                      kv_slot_idx, workspace, status=None, stream=None) -> None:
    i32, dt = torch.int32, cfg.torch_dtype
    _check(load_library().wedlm_window_attn(
        ctypes.byref(cfg), _ptr(q, dt, "q"), _ptr(k, dt, "k"), _ptr(v, dt, "v"), _ptr(k_cache, dt, "k_cache"),
        _ptr(v_cache, dt, "v_cache"), _ptr(block_table, i32, "block_table"), _ptr(prefix_len, i32, "prefix_len"),
        _ptr(pos_ids, i32, "pos_ids"), _ptr(out, dt, "out"), _ptr(kv_slot_idx, i32, "kv_slot_idx"),
        _ptr(workspace, None, "workspace"), ctypes.c_size_t(workspace.numel() * workspace.element_size()),
        _ptr(status, i32, "status"), _stream(stream)), "wedlm_window_attn")


def wedlm_kv_append(cfg, k, v, pos_ids, k_cache, v_cache, block_table, prefix_len, count, kv_slot_idx,
                    status=None, stream=None) -> None:
    i32, dt = torch.int32, cfg.torch_dtype
    _check(load_library().wedlm_kv_append(
        ctypes.byref(cfg), _ptr(k, dt, "k"), _ptr(v, dt, "v"), _ptr(pos_ids, i32, "pos_ids"),
        _ptr(k_cache, dt, "k_cache"), _ptr(v_cache, dt, "v_cache"), _ptr(block_table, i32, "block_table"),
        _ptr(prefix_len, i32, "prefix_len"), _ptr(count, i32, "count"), _ptr(kv_slot_idx, i32, "kv_slot_idx"),
        _ptr(status, i32, "status"), _stream(stream)), "wedlm_kv_append")


def wedlm_confidence_workspace_bytes(cfg) -> int:
    return int(load_library().wedlm_confidence_workspace_bytes(ctypes.byref(cfg)))


def wedlm_confidence_commit(cfg, logits, perm, n_filled, n_commit, window_tokens, filled, prefix_len,
                            window_len, remaining_budget, argmax, maxprob, entropy, lse,
                            committed_tokens, committed_count, filled_count, workspace, status=None, stream=None) -> None:
    i32, u8, f32 = torch.int32, torch.uint8, torch.float32
    _check(load_library().wedlm_confidence_commit(
        ctypes.byref(cfg), _ptr(logits, cfg.torch_dtype, "logits"), _ptr(perm, i32, "perm"),
        _ptr(n_filled, i32, "n_filled"), _ptr(n_commit, i32, "n_commit"),
        _ptr(window_tokens, i32, "window_tokens"), _ptr(filled, u8, "filled"), _ptr(prefix_len, i32, "prefix_len"),
        _ptr(window_len, i32, "window_len"), _ptr(remaining_budget, i32, "remaining_budget"),
        _ptr(argmax, i32, "argmax"), _ptr(maxprob, f32, "maxprob"), _ptr(entropy, f32, "entropy"),
        _ptr(lse, f32, "lse"), _ptr(committed_tokens, i32, "committed_tokens"),
        _ptr(committed_count, i32, "committed_count"), _ptr(filled_count, i32, "filled_count"),
        _ptr(workspace, None, "workspace"), ctypes.c_size_t(workspace.numel() * workspace.element_size()),
        _ptr(status, i32, "status"), _stream(stream)), "wedlm_confidence_commit")


def wedlm_lmhead_confidence_workspace_bytes(cfg, hidden: int) -> int:
    return int(load_library().wedlm_lmhead_confidence_workspace_bytes(ctypes.byref(cfg), ctypes.c_int32(hidden)))


def wedlm_lmhead_confidence_commit(cfg, hidden_states, lm_head, tilt_ids, tilt, perm, n_filled, n_commit, window_tokens,
                                   filled, prefix_len, window_len, remaining_budget, argmax, maxprob, entropy, lse,
                                   committed_tokens, committed_count, filled_count, workspace, status=None, stream=None) -> None:
    """Confidence/commit straight from the hidden states [B,W,H] and the output embedding [V,H] (bf16)."""
    i32, u8, f32, bf = torch.int32, torch.uint8, torch.float32, torch.bfloat16
    _check(load_library().wedlm_lmhead_confidence_commit(
        ctypes.byref(cfg), ctypes.c_int32(hidden_states.shape[-1]), _ptr(hidden_states, bf, "hidden_states"),
        _ptr(lm_head, bf, "lm_head"), _ptr(tilt_ids, i32, "tilt_ids"), ctypes.c_float(tilt), _ptr(perm, i32, "perm"),
        _ptr(n_filled, i32, "n_filled"), _ptr(n_commit, i32, "n_commit"), _ptr(window_tokens, i32, "window_tokens"),
        _ptr(filled, u8, "filled"), _ptr(prefix_len, i32, "prefix_len"), _ptr(window_len, i32, "window_len"),
        _ptr(remaining_budget, i32, "remaining_budget"), _ptr(argmax, i32, "argmax"), _ptr(maxprob, f32, "maxprob"),
        _ptr(entropy, f32, "entropy"), _ptr(lse, f32, "lse"), _ptr(committed_tokens, i32, "committed_tokens"),
        _ptr(committed_count, i32, "committed_count"), _ptr(filled_count, i32, "filled_count"),
        _ptr(workspace, None, "workspace"), ctypes.c_size_t(workspace.numel() * workspace.element_size()),
        _ptr(status, i32, "status"), _stream(stream)), "wedlm_lmhead_confidence_commit")


WEDLM_STATIC_SCRATCH_BYTES = 4 << 20
WEDLM_ERR_STATIC_SCRATCH = -6


def wedlm_confidence_commit_static(cfg, logits, perm, n_filled, n_commit, window_tokens, filled, prefix_len,
                                   window_len, remaining_budget, argmax, maxprob, entropy, lse,
                                   committed_tokens, committed_count, filled_count, status=None, stream=None) -> None:
    """wedlm_confidence_commit for callers that may not allocate device memory (a process whose HBM is
    already committed to a cache pool, a loop that bans allocator calls): same inputs and outputs, no
    workspace; the scratch is a fixed 4 MiB array inside the library.  Raises WedlmError with code
    WEDLM_ERR_STATIC_SCRATCH when batch*window*chunks does not fit.  Calls that may overlap on the GPU
    must be serialised by the caller; the first call on a device should precede any stream capture."""
    i32, u8, f32 = torch.int32, torch.uint8, torch.float32
    _check(load_library().wedlm_confidence_commit_static(
        ctypes.byref(cfg), _ptr(logits, cfg.torch_dtype, "logits"), _ptr(perm, i32, "perm"),
        _ptr(n_filled, i32, "n_filled"), _ptr(n_commit, i32, "n_commit"),
        _ptr(window_tokens, i32, "window_tokens"), _ptr(filled, u8, "filled"), _ptr(prefix_len, i32, "prefix_len"),
        _ptr(window_len, i32, "window_len"), _ptr(remaining_budget, i32, "remaining_budget"),
        _ptr(argmax, i32, "argmax"), _ptr(maxprob, f32, "maxprob"), _ptr(entropy, f32, "entropy"),
        _ptr(lse, f32, "lse"), _ptr(committed_tokens, i32, "committed_tokens"),
        _ptr(committed_count, i32, "committed_count"), _ptr(filled_count, i32, "filled_count"),
        _ptr(status, i32, "status"), _stream(stream)), "wedlm_confidence_commit_static")


def wedlm_window_refill(cfg, n_commit, window_tokens, filled, prefix_len, window_len, remaining_budget,
                        committed_tokens, committed_count, stream=None) -> None:
    i32, u8 = torch.int32, torch.uint8
    _check(load_library().wedlm_window_refill(
        ctypes.byref(cfg), _ptr(n_commit, i32, "n_commit"), _ptr(window_tokens, i32, "window_tokens"),
        _ptr(filled, u8, "filled"), _ptr(prefix_len, i32, "prefix_len"), _ptr(window_len, i32, "window_len"),
        _ptr(remaining_budget, i32, "remaining_budget"), _ptr(committed_tokens, i32, "committed_tokens"),
        _ptr(committed_count, i32, "committed_count"), _stream(stream)), "wedlm_window_refill")


def _hptr(t: Optional[torch.Tensor], dtype: Optional[torch.dtype], name: str):
    """Host tensor -> raw pointer (page-locked memory is the caller's business)."""
    if t is None:
        return None
    if not isinstance(t, torch.Tensor) or t.is_cuda:
        raise TypeError(f"{name} must be a CPU tensor")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name} must have dtype {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    return ctypes.c_void_p(t.data_ptr())


def wedlm_step_host_workspace_bytes(cfg) -> int:
    return int(load_library().wedlm_step_host_workspace_bytes(ctypes.byref(cfg)))


def wedlm_step_host(cfg, h_filled, h_window_tokens, h_prefix_len, h_window_len, h_remaining_budget, h_block_table,
                    h_q, h_k, h_v, h_logits, k_cache, v_cache, h_committed_tokens, h_committed_count, h_filled_count,
                    workspace, status=None, stream=None) -> int:
    """One whole step from host tensors (bf16 tensors may be passed as int16/uint16 bit patterns).  Asynchronous
    on the stream.  Returns the device address of the attention output inside the workspace."""
    i32, u8 = torch.int32, torch.uint8
    out_ptr = ctypes.c_void_p()
    _check(load_library().wedlm_step_host(
        ctypes.byref(cfg), _hptr(h_filled, u8, "h_filled"), _hptr(h_window_tokens, i32, "h_window_tokens"),
        _hptr(h_prefix_len, i32, "h_prefix_len"), _hptr(h_window_len, i32, "h_window_len"),
        _hptr(h_remaining_budget, i32, "h_remaining_budget"), _hptr(h_block_table, i32, "h_block_table"),
        _hptr(h_q, None, "h_q"), _hptr(h_k, None, "h_k"), _hptr(h_v, None, "h_v"), _hptr(h_logits, None, "h_logits"),
        _ptr(k_cache, cfg.torch_dtype, "k_cache"), _ptr(v_cache, cfg.torch_dtype, "v_cache"),
        _hptr(h_committed_tokens, i32, "h_committed_tokens"), _hptr(h_committed_count, i32, "h_committed_count"),
        _hptr(h_filled_count, i32, "h_filled_count"), _ptr(workspace, None, "workspace"),
        ctypes.c_size_t(workspace.numel() * workspace.element_size()), ctypes.byref(out_ptr),
        _ptr(status, i32, "status"), _stream(stream)), "wedlm_step_host")
    return int(out_ptr.value or 0)


def wedlm_step_host_lmhead_workspace_bytes(cfg, hidden: int) -> int:
    return int(load_library().wedlm_step_host_lmhead_workspace_bytes(ctypes.byref(cfg), ctypes.c_int32(hidden)))


def wedlm_step_host_lmhead(cfg, h_filled, h_window_tokens, h_prefix_len, h_window_len, h_remaining_budget, h_block_table,
                           h_q, h_k, h_v, h_hidden_states, lm_head, h_tilt_ids, tilt, k_cache, v_cache, h_committed_tokens,
                           h_committed_count, h_filled_count, workspace, status=None, stream=None) -> int:
    """One whole step from host tensors with the LM head inside it: hidden states [B,W,H] come from the host, the
    output embedding [V,H] is a device tensor.  Returns the device address of the attention output."""
    i32, u8 = torch.int32, torch.uint8
    out_ptr = ctypes.c_void_p()
    _check(load_library().wedlm_step_host_lmhead(
        ctypes.byref(cfg), ctypes.c_int32(h_hidden_states.shape[-1]), _hptr(h_filled, u8, "h_filled"),
        _hptr(h_window_tokens, i32, "h_window_tokens"), _hptr(h_prefix_len, i32, "h_prefix_len"),
        _hptr(h_window_len, i32, "h_window_len"), _hptr(h_remaining_budget, i32, "h_remaining_budget"),
        _hptr(h_block_table, i32, "h_block_table"), _hptr(h_q, None, "h_q"), _hptr(h_k, None, "h_k"), _hptr(h_v, None, "h_v"),
        _hptr(h_hidden_states, None, "h_hidden_states"), _ptr(lm_head, torch.bfloat16, "lm_head"),
        _hptr(h_tilt_ids, i32, "h_tilt_ids"), ctypes.c_float(tilt), _ptr(k_cache, cfg.torch_dtype, "k_cache"),
        _ptr(v_cache, cfg.torch_dtype, "v_cache"), _hptr(h_committed_tokens, i32, "h_committed_tokens"),
        _hptr(h_committed_count, i32, "h_committed_count"), _hptr(h_filled_count, i32, "h_filled_count"),
        _ptr(workspace, None, "workspace"), ctypes.c_size_t(workspace.numel() * workspace.element_size()),
        ctypes.byref(out_ptr), _ptr(status, i32, "status"), _stream(stream)), "wedlm_step_host_lmhead")
    return int(out_ptr.value or 0)


def wedlm_dual_stream_construct(cfg, n_blocks, seq_len, tokens, masked, x_input, p_input, is_mask=None, n_observed=None,
                                stream=None) -> None:
    i32, u8 = torch.int32, torch.uint8
    _check(load_library().wedlm_dual_stream_construct(
        ctypes.byref(cfg), ctypes.c_int32(n_blocks), ctypes.c_int32(seq_len), _ptr(tokens, i32, "tokens"),
        _ptr(masked, u8, "masked"), _ptr(x_input, i32, "x_input"), _ptr(p_input, i32, "p_input"),
        _ptr(is_mask, u8, "is_mask"), _ptr(n_observed, i32, "n_observed"), _stream(stream)), "wedlm_dual_stream_construct")


def wedlm_dual_stream_workspace_bytes(cfg, n_blocks) -> int:
    return int(load_library().wedlm_dual_stream_workspace_bytes(ctypes.byref(cfg), ctypes.c_int32(n_blocks)))


def wedlm_dual_stream_attn(cfg, n_blocks, q, k, v, p_input, out, workspace, status=None, stream=None) -> None:
    dt = cfg.torch_dtype
    _check(load_library().wedlm_dual_stream_attn(
        ctypes.byref(cfg), ctypes.c_int32(n_blocks), _ptr(q, dt, "q"), _ptr(k, dt, "k"), _ptr(v, dt, "v"),
        _ptr(p_input, torch.int32, "p_input"), _ptr(out, dt, "out"), _ptr(workspace, None, "workspace"),
        ctypes.c_size_t(workspace.numel() * workspace.element_size()), _ptr(status, torch.int32, "status"),
        _stream(stream)), "wedlm_dual_stream_attn")


# ----------------------------------------------------------------------------------------
# one decoding step with preallocated buffers (allocation + call order only)
# ----------------------------------------------------------------------------------------
def to_device(x: np.ndarray, device="cuda") -> torch.Tensor:
    """numpy -> CUDA tensor; uint16 arrays are bf16 bit patterns."""
    if x.dtype == np.uint16:
        return torch.from_numpy(x.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(x)).to(device)


class DecodeStep:
    """Owns the outputs and workspaces of one step for a fixed config and runs the three calls
    reorder -> window attention -> confidence/commit on the current stream."""

    def __init__(self, cfg: WedlmConfig, device="cuda"):
        load_library()
        self.cfg = cfg
        B, W = cfg.batch, cfg.window
        i32 = dict(dtype=torch.int32, device=device)
        f32 = dict(dtype=torch.float32, device=device)
        self.perm = torch.empty(B, W, **i32)
        self.inv_perm = torch.empty(B, W, **i32)
        self.pos_ids = torch.empty(B, W, **i32)
        self.tokens_phys = torch.empty(B, W, **i32)
        self.n_filled = torch.empty(B, **i32)
        self.n_commit = torch.empty(B, **i32)
        self.out = torch.empty(B, W, cfg.n_q_heads, cfg.head_dim, dtype=cfg.torch_dtype, device=device)
        self.kv_slot_idx = torch.empty(B, W, **i32)
        self.status = torch.zeros(1, **i32)
        self.attn_ws = torch.empty(max(wedlm_window_attn_workspace_bytes(cfg), 256), dtype=torch.uint8, device=device)
        self.conf_ws = torch.empty(max(wedlm_confidence_workspace_bytes(cfg), 256), dtype=torch.uint8, device=device)
        self.argmax = torch.empty(B, W, **i32)
        self.maxprob = torch.empty(B, W, **f32)
        self.entropy = torch.empty(B, W, **f32)
        self.lse = torch.empty(B, W, **f32)
        self.committed_tokens = torch.empty(B, W, **i32)
        self.committed_count = torch.empty(B, **i32)
        self.filled_count = torch.empty(B, **i32)

    def reorder(self, filled, window_tokens, prefix_len, window_len=None):
        wedlm_reorder(self.cfg, filled, window_tokens, prefix_len, window_len, self.perm, self.inv_perm,
                      self.pos_ids, self.tokens_phys, self.n_filled, self.n_commit)

    def attention(self, q, k, v, k_cache, v_cache, block_table, prefix_len):
        wedlm_window_attn(self.cfg, q, k, v, k_cache, v_cache, block_table, prefix_len, self.pos_ids, self.out,
                          self.kv_slot_idx, self.attn_ws, self.status)

    def confidence_commit(self, logits, window_tokens, filled, prefix_len, window_len=None, remaining_budget=None):
        wedlm_confidence_commit(self.cfg, logits, self.perm, self.n_filled, self.n_commit, window_tokens, filled,
                                prefix_len, window_len, remaining_budget, self.argmax, self.maxprob, self.entropy,
                                self.lse, self.committed_tokens, self.committed_count, self.filled_count,
                                self.conf_ws, self.status)

    def capture_graph(self, d: Dict[str, torch.Tensor], window_len=None, remaining_budget=None) -> "torch.cuda.CUDAGraph":
        """Capture reorder -> attention -> confidence/commit on these fixed buffers into a CUDA graph.
        The calls are asynchronous and read their sizes from device memory, so one capture serves
        every later step: replaying it advances the device-resident window state again.  One
        un-captured run comes first (it performs the per-device set-up)."""
        self.run(d, window_len, remaining_budget)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            self.run(d, window_len, remaining_budget)
        return graph

    def run(self, d: Dict[str, torch.Tensor], window_len=None, remaining_budget=None) -> None:
        """d holds device tensors named as in workloads.make_step(); window state is updated in place."""
        self.reorder(d["filled"], d["window_tokens"], d["prefix_len"], window_len)
        self.attention(d["q"], d["k"], d["v"], d["k_cache"], d["v_cache"], d["block_table"], d["prefix_len"])
        self.confidence_commit(d["logits"], d["window_tokens"], d["filled"], d["prefix_len"], window_len,
                               remaining_budget)


def config_for(step_cfg, *, max_pages_per_seq: int, num_pages: int, max_prefix_len: int,
               attn_impl: str = "auto", batch: Optional[int] = None, commit_mode: str = "streaming",
               sample_temperature: float = 0.0, sample_seed: int = 0) -> WedlmConfig:
    """wedlm_config_t for an object with the attribute names of a workload description
    (batch, window, n_q_heads, n_kv_heads, head_dim, page_size, vocab, dtype, rope_theta,
    conf_mode, tau, lam, maxprob_thr, mask_token_id)."""
    return make_config(
        batch=step_cfg.batch if batch is None else batch, window=step_cfg.window,
        n_q_heads=step_cfg.n_q_heads, n_kv_heads=step_cfg.n_kv_heads, head_dim=step_cfg.head_dim,
        page_size=step_cfg.page_size, max_pages_per_seq=max_pages_per_seq, num_pages=num_pages,
        vocab=step_cfg.vocab, dtype=step_cfg.dtype, rope_theta=step_cfg.rope_theta,
        conf_mode=step_cfg.conf_mode, tau=step_cfg.tau, lam=step_cfg.lam, maxprob_thr=step_cfg.maxprob_thr,
        mask_token_id=step_cfg.mask_token_id, max_prefix_len=max_prefix_len, attn_impl=attn_impl,
        commit_mode=commit_mode, sample_temperature=sample_temperature, sample_seed=sample_seed)
