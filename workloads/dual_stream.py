"""Seeded inputs of a Dual-Stream Masking training forward (Section 4.2): token ids, which logical
positions of the prediction stream are masked, and random q / k / v for the 2 x L physical rows.

Data only: no reordering, no positions, no mask logic and no attention live here.  Masked positions
follow the paper's recipe: the prediction stream is cut into blocks of B tokens, each block draws its
own masking ratio gamma_k uniformly from (0, 1] and masks ceil(gamma_k * block_len) positions chosen
uniformly without replacement."""
from __future__ import annotations

import dataclasses
from typing import Dict

import numpy as np

from .synth import BASE_SEED, bf16_bits


@dataclasses.dataclass(frozen=True)
class DualStreamConfig:
    name: str
    n_seq: int                 # sequences
    seq_len: int               # L tokens per stream
    block: int                 # B
    n_q_heads: int = 32
    n_kv_heads: int = 8
    head_dim: int = 128
    vocab: int = 151936
    dtype: str = "bf16"
    rope_theta: float = 1.0e6
    page_size: int = 16

    @property
    def mask_token_id(self) -> int:
        return self.vocab - 1

    @property
    def n_blocks(self) -> int:
        return (self.seq_len + self.block - 1) // self.block

    @property
    def padded_len(self) -> int:
        return self.n_blocks * self.block

    def replace(self, **kw) -> "DualStreamConfig":
        return dataclasses.replace(self, **kw)


DS_CONFIGS: Dict[str, DualStreamConfig] = {
    # small enough for the dense fp64 oracle, several blocks and a ragged last one
    "ds_small": DualStreamConfig(name="ds_small", n_seq=2, seq_len=150, block=32),
    # the paper's block size on a 4k context of Qwen3-8B attention geometry
    "ds_4k": DualStreamConfig(name="ds_4k", n_seq=1, seq_len=4096, block=32),
    "ds_8k": DualStreamConfig(name="ds_8k", n_seq=1, seq_len=8192, block=32),
}


def _g(seed: int, sub: int) -> np.random.Generator:
    return np.random.Generator(np.random.SFC64(np.random.SeedSequence([seed, 3000, sub])))


def make_dual_stream(cfg: DualStreamConfig, seed: int = BASE_SEED) -> Dict[str, np.ndarray]:
    """tokens i32 [N, L]; masked u8 [N, L] (logical order); gamma f32 [N, K];
    q [N, 2, Lp, Hq, D], k, v [N, 2, Lp, Hkv, D] in physical order (stream 0 = memory, 1 = prediction;
    Lp = K * B, rows at or beyond L are padding), stored as bf16 bit patterns or fp32."""
    N, L, B, K, Lp = cfg.n_seq, cfg.seq_len, cfg.block, cfg.n_blocks, cfg.padded_len
    g = _g(seed, 0)
    tokens = g.integers(0, cfg.vocab - 1, size=(N, L)).astype(np.int32)
    masked = np.zeros((N, L), np.uint8)
    gamma = np.zeros((N, K), np.float32)
    for n in range(N):
        for kb in range(K):
            lo, hi = kb * B, min((kb + 1) * B, L)
            gm = 1.0 - g.random()                      # uniform on (0, 1]
            gamma[n, kb] = gm
            cnt = int(np.ceil(gm * (hi - lo)))
            masked[n, lo + g.choice(hi - lo, size=cnt, replace=False)] = 1

    def tensor(sub: int, heads: int) -> np.ndarray:
        x = _g(seed, sub).standard_normal((N, 2, Lp, heads, cfg.head_dim), dtype=np.float32)
        return bf16_bits(x.reshape(-1)).reshape(x.shape) if cfg.dtype == "bf16" else x

    return dict(tokens=tokens, masked=masked, gamma=gamma, q=tensor(1, cfg.n_q_heads), k=tensor(2, cfg.n_kv_heads),
                v=tensor(3, cfg.n_kv_heads))
