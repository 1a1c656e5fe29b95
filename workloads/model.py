"""Seeded random-init decoder weights, prompts and target sequences for the decoding-loop harness.

Data only: the arrays drawn here are consumed by the GPU loop (paper_2512_22737_b200/loop.py) and
by the fp64 oracle model (oracle/model_oracle.py); neither the forward pass nor any decoding logic
lives in this file."""
from __future__ import annotations

import dataclasses
from typing import Dict

import numpy as np

from .synth import BASE_SEED, bf16_bits


@dataclasses.dataclass(frozen=True)
class ModelConfig:
    """Pre-norm decoder with RMSNorm, GQA attention with RoPE and a SwiGLU MLP (Qwen-style layout;
    no QK-norm, no biases)."""
    name: str
    vocab: int
    hidden: int
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    dtype: str = "f32"              # "f32" | "bf16": storage type of weights and activations
    rope_theta: float = 1.0e6
    rms_eps: float = 1.0e-6
    init_std: float = 0.02

    @property
    def mask_token_id(self) -> int:
        return self.vocab - 1


TINY = ModelConfig(name="tiny", vocab=1001, hidden=64, n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=32,
                   ffn=128, dtype="f32", rope_theta=1.0e4, init_std=0.25)

# Four layers of Qwen3-8B width.
QWEN_4L = ModelConfig(name="qwen3_8b_width_4l", vocab=151936, hidden=4096, n_layers=4, n_q_heads=32, n_kv_heads=8,
                      head_dim=128, ffn=12288, dtype="bf16", rope_theta=1.0e6, init_std=0.02)


def _store(x: np.ndarray, dtype: str) -> np.ndarray:
    return bf16_bits(x.reshape(-1)).reshape(x.shape) if dtype == "bf16" else x.astype(np.float32)


def make_model(cfg: ModelConfig, seed: int = BASE_SEED) -> Dict[str, np.ndarray]:
    """N(0, init_std^2) matrices, unit norm gains.  bf16 models are returned as uint16 bit patterns.

    Keys: embed [V,H], lm_head [H,V], norm_f [H]; per layer l: l{l}.norm1, l{l}.norm2 [H],
    l{l}.wq [H,Hq*D], l{l}.wk, l{l}.wv [H,Hkv*D], l{l}.wo [Hq*D,H], l{l}.wg, l{l}.wu [H,F], l{l}.wd [F,H]."""
    w: Dict[str, np.ndarray] = {}

    def mat(name, shape, sub):
        g = np.random.Generator(np.random.SFC64(np.random.SeedSequence([seed, 1000, sub])))
        w[name] = _store(g.standard_normal(shape, dtype=np.float32) * np.float32(cfg.init_std), cfg.dtype)

    H, F = cfg.hidden, cfg.ffn
    mat("embed", (cfg.vocab, H), 0)
    mat("lm_head", (H, cfg.vocab), 1)
    w["norm_f"] = _store(np.ones(H, np.float32), cfg.dtype)
    for l in range(cfg.n_layers):
        w[f"l{l}.norm1"] = _store(np.ones(H, np.float32), cfg.dtype)
        w[f"l{l}.norm2"] = _store(np.ones(H, np.float32), cfg.dtype)
        mat(f"l{l}.wq", (H, cfg.n_q_heads * cfg.head_dim), 10 * l + 2)
        mat(f"l{l}.wk", (H, cfg.n_kv_heads * cfg.head_dim), 10 * l + 3)
        mat(f"l{l}.wv", (H, cfg.n_kv_heads * cfg.head_dim), 10 * l + 4)
        mat(f"l{l}.wo", (cfg.n_q_heads * cfg.head_dim, H), 10 * l + 5)
        mat(f"l{l}.wg", (H, F), 10 * l + 6)
        mat(f"l{l}.wu", (H, F), 10 * l + 7)
        mat(f"l{l}.wd", (F, H), 10 * l + 8)
    return w


def make_prompts_and_targets(cfg: ModelConfig, batch: int, prompt_len: int, new_tokens: int,
                             seed: int = BASE_SEED) -> Dict[str, np.ndarray]:
    """prompt i32 [B, prompt_len]; target i32 [B, prompt_len + new_tokens]: the token the logits are
    tilted toward at each absolute position (ids below the mask id)."""
    g = np.random.Generator(np.random.SFC64(np.random.SeedSequence([seed, 2000])))
    prompt = g.integers(0, cfg.vocab - 1, size=(batch, prompt_len)).astype(np.int32)
    target = g.integers(0, cfg.vocab - 1, size=(batch, prompt_len + new_tokens)).astype(np.int32)
    return dict(prompt=prompt, target=target)
