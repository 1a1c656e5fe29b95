"""Seeded generators for the step inputs (data only, no method arithmetic)."""
from __future__ import annotations

import dataclasses
import os
from concurrent.futures import ThreadPoolExecutor
from typing import Dict, Optional

import numpy as np

BASE_SEED = 251222737

# Named random streams: every tensor draws from its own stream so that adding a
# tensor never shifts the values of another.
_STREAMS = {
    "prefix_len": 1, "obs_prob": 2, "filled": 3, "tokens": 4, "pages": 5,
    "k_cache": 6, "v_cache": 7, "q": 8, "k": 9, "v": 10,
    "logits": 11, "boost_rows": 12, "targets": 13,
}


@dataclasses.dataclass(frozen=True)
class StepConfig:
    """Shapes and distributions of one synthetic decoding step."""
    name: str
    batch: int
    window: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    vocab: int
    dtype: str = "bf16"            # "bf16" | "f32": storage type of q/k/v, cache and logits
    page_size: int = 16
    prefix_lo: int = 0             # committed prefix length ~ U{prefix_lo..prefix_hi}
    prefix_hi: int = 0
    obs_prob_lo: float = 0.5       # per-sequence probability that a slot is filled
    obs_prob_hi: float = 0.5
    obs_pattern: str = "bernoulli"  # "bernoulli" | "runs" (alternating geometric runs)
    obs_run_mean: float = 4.0
    rope_theta: float = 1.0e6
    conf_mode: str = "entropy"     # "entropy": H + lambda*d <= tau ; "maxprob": p_max >= thr
    tau: float = 0.3
    lam: float = 0.10
    maxprob_thr: float = 0.9
    logit_sigma: float = 1.0
    boost: float = 8.0             # added to the target id's logit on boosted rows
    boost_prob: float = 0.5        # fraction of rows that carry a boosted target
    spare_pages: int = 3

    @property
    def mask_token_id(self) -> int:
        return self.vocab - 1

    def replace(self, **kw) -> "StepConfig":
        return dataclasses.replace(self, **kw)


_QWEN = dict(n_q_heads=32, n_kv_heads=8, head_dim=128, vocab=151936, dtype="bf16",
             rope_theta=1.0e6, conf_mode="entropy", tau=0.3, lam=0.10)

CONFIGS: Dict[str, StepConfig] = {
    # Tiny single-layer step the CPU oracle finishes at once.
    "cfg1_tiny": StepConfig(
        name="cfg1_tiny", batch=1, window=8, n_q_heads=4, n_kv_heads=2, head_dim=64,
        vocab=1001, dtype="f32", prefix_lo=64, prefix_hi=64, obs_prob_lo=0.4, obs_prob_hi=0.4,
        rope_theta=1.0e4, conf_mode="maxprob", maxprob_thr=0.9, logit_sigma=3.0,
        boost=0.0, boost_prob=0.0),
    # Qwen3-8B-shaped single layer, one sequence.
    "cfg2_qwen_b1": StepConfig(
        name="cfg2_qwen_b1", batch=1, window=16, prefix_lo=2048, prefix_hi=2048,
        obs_prob_lo=0.3, obs_prob_hi=0.3, boost=8.0, boost_prob=0.5, **_QWEN),
    # Batched serving step with ragged prefixes.
    "cfg3_batched": StepConfig(
        name="cfg3_batched", batch=64, window=32, prefix_lo=512, prefix_hi=8192,
        obs_prob_lo=0.1, obs_prob_hi=0.6, boost=8.0, boost_prob=0.7, **_QWEN),
    # Long-context step, clustered observed runs.
    "cfg4_long": StepConfig(
        name="cfg4_long", batch=8, window=64, prefix_lo=32768, prefix_hi=32768,
        obs_prob_lo=0.5, obs_prob_hi=0.5, obs_pattern="runs", obs_run_mean=4.0,
        boost=8.0, boost_prob=0.9, **_QWEN),
}


def get_config(name: str) -> StepConfig:
    return CONFIGS[name]


# ----------------------------------------------------------------------------------------
# bf16 bit patterns (storage format conversion only)
# ----------------------------------------------------------------------------------------
def bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit pattern (uint16), round-to-nearest-even.  Finite inputs only."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) >> np.uint32(16)).astype(np.uint16)


def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    """bf16 bit pattern (uint16) -> the fp32 value it denotes (exact)."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


# ----------------------------------------------------------------------------------------
# random helpers
# ----------------------------------------------------------------------------------------
def _rng(seed: int, stream: str, sub: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.SFC64(np.random.SeedSequence([seed, _STREAMS[stream], sub])))


_CHUNK = 1 << 22  # elements per independently seeded chunk (result does not depend on thread count)


def _normal_store(n: int, seed: int, stream: str, sigma: float, dtype: str) -> np.ndarray:
    """n i.i.d. N(0, sigma^2) values, generated in fp32, stored as fp32 or as bf16 bit patterns."""
    out = np.empty(n, dtype=np.uint16 if dtype == "bf16" else np.float32)
    n_chunks = (n + _CHUNK - 1) // _CHUNK

    def work(c: int) -> None:
        lo, hi = c * _CHUNK, min(n, (c + 1) * _CHUNK)
        x = _rng(seed, stream, c).standard_normal(hi - lo, dtype=np.float32)
        if sigma != 1.0:
            x *= np.float32(sigma)
        out[lo:hi] = bf16_bits(x) if dtype == "bf16" else x

    workers = min(n_chunks, max(1, len(os.sched_getaffinity(0))))
    if workers <= 1:
        for c in range(n_chunks):
            work(c)
    else:
        with ThreadPoolExecutor(max_workers=workers) as ex:
            list(ex.map(work, range(n_chunks)))
    return out


def _filled_pattern(cfg: StepConfig, seed: int, prob: np.ndarray) -> np.ndarray:
    B, W = cfg.batch, cfg.window
    g = _rng(seed, "filled")
    if cfg.obs_pattern == "bernoulli":
        return (g.random((B, W)) < prob[:, None]).astype(np.uint8)
    # Alternating renewal process: observed runs and mask runs, both geometric with the given
    # mean; the first run is observed with the sequence's observed probability.
    out = np.zeros((B, W), dtype=np.uint8)
    p_stop = 1.0 / cfg.obs_run_mean
    for b in range(B):
        state = 1 if g.random() < prob[b] else 0
        j = 0
        while j < W:
            run = int(g.geometric(p_stop))
            out[b, j:j + run] = state
            j += run
            state ^= 1
    return out


def make_step(cfg: StepConfig, seed: int = BASE_SEED, *, with_logits: bool = True,
              prefix_len: Optional[np.ndarray] = None,
              filled: Optional[np.ndarray] = None) -> Dict[str, np.ndarray]:
    """Draw every input of one decoding step.

    Returns a dict of numpy arrays (bf16 tensors as uint16 bit patterns):
      filled          u8  [B,W]   logical order; 1 = slot holds a predicted, uncommitted token
      window_tokens   i32 [B,W]   logical order; mask slots hold cfg.mask_token_id
      prefix_len      i32 [B]     committed prefix length P_b
      block_table     i32 [B,max_pages]  physical page of each logical page (-1 where unused)
      k_cache,v_cache     [num_pages,Hkv,page,D]   already-rotated K and V of the prefix
      q,k,v               [B,W,H,D]   window projections, physical order, before RoPE
      logits              [B,W,V]     physical order
      targets         i32 [B,W]   boosted token id of each physical row (-1 if not boosted)
    `prefix_len` / `filled` override the drawn values (edge-case tests).
    """
    B, W, Hq, Hkv, D, pg = cfg.batch, cfg.window, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.page_size
    V = cfg.vocab
    out: Dict[str, np.ndarray] = {}

    if prefix_len is None:
        prefix_len = _rng(seed, "prefix_len").integers(cfg.prefix_lo, cfg.prefix_hi + 1, size=B)
    prefix_len = np.asarray(prefix_len, dtype=np.int32)
    prob = _rng(seed, "obs_prob").uniform(cfg.obs_prob_lo, cfg.obs_prob_hi, size=B)
    if filled is None:
        filled = _filled_pattern(cfg, seed, prob)
    filled = np.asarray(filled, dtype=np.uint8)
    tok = _rng(seed, "tokens").integers(0, V - 1, size=(B, W)).astype(np.int32)
    tok[filled == 0] = cfg.mask_token_id
    out.update(filled=filled, window_tokens=tok, prefix_len=prefix_len)

    # Paged cache: each sequence owns ceil((P+W)/page) pages, scattered over the pool by a
    # seeded permutation (a fragmented live cache).
    pages_per_seq = (prefix_len.astype(np.int64) + W + pg - 1) // pg
    max_pages = int(pages_per_seq.max())
    num_pages = int(pages_per_seq.sum()) + cfg.spare_pages
    order = _rng(seed, "pages").permutation(num_pages).astype(np.int32)
    table = np.full((B, max_pages), -1, dtype=np.int32)
    at = 0
    for b in range(B):
        n = int(pages_per_seq[b])
        table[b, :n] = order[at:at + n]
        at += n
    out["block_table"] = table
    n_cache = num_pages * Hkv * pg * D
    shape_c = (num_pages, Hkv, pg, D)
    out["k_cache"] = _normal_store(n_cache, seed, "k_cache", 1.0, cfg.dtype).reshape(shape_c)
    out["v_cache"] = _normal_store(n_cache, seed, "v_cache", 1.0, cfg.dtype).reshape(shape_c)
    out["q"] = _normal_store(B * W * Hq * D, seed, "q", 1.0, cfg.dtype).reshape(B, W, Hq, D)
    out["k"] = _normal_store(B * W * Hkv * D, seed, "k", 1.0, cfg.dtype).reshape(B, W, Hkv, D)
    out["v"] = _normal_store(B * W * Hkv * D, seed, "v", 1.0, cfg.dtype).reshape(B, W, Hkv, D)

    boosted = _rng(seed, "boost_rows").random((B, W)) < cfg.boost_prob
    targets = _rng(seed, "targets").integers(0, V - 1, size=(B, W)).astype(np.int32)
    targets[~boosted] = -1
    out["targets"] = targets
    if with_logits:
        out["logits"] = _logits(cfg, seed, targets)
    return out


def _logits(cfg: StepConfig, seed: int, targets: np.ndarray) -> np.ndarray:
    """[B,W,V] rows of N(0, sigma^2) with `boost` added on each row's target id.

    Drawn in fp32, boosted in fp32, rounded once to the storage type; one independently seeded
    stream per sequence, so the result does not depend on the thread count."""
    B, W, V = cfg.batch, cfg.window, cfg.vocab
    logits = np.empty((B, W, V), dtype=np.uint16 if cfg.dtype == "bf16" else np.float32)

    def work(b: int) -> None:
        x = _rng(seed, "logits", b).standard_normal((W, V), dtype=np.float32)
        if cfg.logit_sigma != 1.0:
            x *= np.float32(cfg.logit_sigma)
        rows = np.nonzero(targets[b] >= 0)[0]
        x[rows, targets[b, rows]] += np.float32(cfg.boost)
        logits[b] = bf16_bits(x.reshape(-1)).reshape(W, V) if cfg.dtype == "bf16" else x

    workers = min(B, max(1, len(os.sched_getaffinity(0))))
    if workers <= 1:
        for b in range(B):
            work(b)
    else:
        with ThreadPoolExecutor(max_workers=workers) as ex:
            list(ex.map(work, range(B)))
    return logits
