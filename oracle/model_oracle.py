"""fp64 oracle of the decoding-loop harness: a cache-free transformer forward plus Algorithm 1.

TEST INFRASTRUCTURE ONLY (same rules as wedlm_oracle.py: imported by tests and the benchmark's CPU
leg, shares nothing with the CUDA path).

The point of this file is independence from every caching trick: each forward recomputes the whole
sequence (committed text followed by the reordered window) from the token ids in float64, under
the visibility the method states (Section 4.1 and 5.2): a committed token sees the committed tokens
before it and itself; window row i (physical order) sees all committed tokens and window rows
j <= i; RoPE uses each token's logical position id (Section 2.2).  If the GPU loop's paged cache,
in-place commit or staging were wrong, its text would diverge from this one.
"""
from __future__ import annotations

from typing import Dict, List, Sequence

import numpy as np

from . import wedlm_oracle as orc


def _rms(x: np.ndarray, gain: np.ndarray, eps: float) -> np.ndarray:
    return x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps) * gain


def _silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def forward_window(weights: Dict[str, np.ndarray], mcfg, committed: Sequence[int], tokens_phys: Sequence[int],
                   pos_ids: Sequence[int]) -> np.ndarray:
    """Logits [len(tokens_phys), V] of the window rows.  `committed` are the tokens at positions
    0..P-1; the window rows carry their own position ids."""
    w = {k: orc.to_f64(v) for k, v in weights.items()}
    P, Wn = len(committed), len(tokens_phys)
    N = P + Wn
    toks = np.asarray(list(committed) + list(tokens_phys), dtype=np.int64)
    pos = np.asarray(list(range(P)) + list(pos_ids), dtype=np.int64)
    # visibility: row a may look at column c
    vis = np.zeros((N, N), dtype=bool)
    for a in range(N):
        if a < P:
            vis[a, : a + 1] = True
        else:
            vis[a, :P] = True
            vis[a, P: a + 1] = True           # window rows j <= i in physical order
    Hq, Hkv, D = mcfg.n_q_heads, mcfg.n_kv_heads, mcfg.head_dim
    G = Hq // Hkv
    scale = 1.0 / np.sqrt(D)
    h = w["embed"][toks]
    for l in range(mcfg.n_layers):
        a = _rms(h, w[f"l{l}.norm1"], mcfg.rms_eps)
        q = (a @ w[f"l{l}.wq"]).reshape(N, Hq, D)
        k = (a @ w[f"l{l}.wk"]).reshape(N, Hkv, D)
        v = (a @ w[f"l{l}.wv"]).reshape(N, Hkv, D)
        q = orc.rope(q, pos[:, None], mcfg.rope_theta)
        k = orc.rope(k, pos[:, None], mcfg.rope_theta)
        out = np.zeros((N, Hq, D))
        for hh in range(Hq):
            s = scale * (q[:, hh] @ k[:, hh // G].T)
            s = np.where(vis, s, -np.inf)
            p = np.exp(s - s.max(axis=1, keepdims=True))
            p /= p.sum(axis=1, keepdims=True)
            out[:, hh] = p @ v[:, hh // G]
        h = h + out.reshape(N, Hq * D) @ w[f"l{l}.wo"]
        m = _rms(h, w[f"l{l}.norm2"], mcfg.rms_eps)
        h = h + (_silu(m @ w[f"l{l}.wg"]) * (m @ w[f"l{l}.wu"])) @ w[f"l{l}.wd"]
    logits = _rms(h, w["norm_f"], mcfg.rms_eps) @ w["lm_head"]
    return logits[P:]


def decode(weights, mcfg, prompt: Sequence[int], target: Sequence[int], *, tilt: float, window: int,
           max_new_tokens: int, conf_mode: str, tau: float, lam: float, maxprob_thr: float,
           block_commit: bool = False, temperature: float = 0.0, sample_seed=(0, 0),
           seq_index: int = 0) -> Dict[str, object]:
    """Algorithm 1 for one sequence on the model above; logits[row, target[position of row]] += tilt.
    With temperature > 0 the filled tokens are draws (keyed by sample_seed, seq_index and position)."""
    prompt = [int(t) for t in prompt]

    def forward(y: List[int], toks: List[int], pos: List[int]) -> np.ndarray:
        lg = forward_window(weights, mcfg, prompt + y, toks, pos)
        if tilt != 0.0:
            for r, pp in enumerate(pos):
                lg[r, int(target[min(pp, len(target) - 1)])] += tilt
        return lg

    return orc.decode_loop(forward, prefix_len=len(prompt), window=window, max_new_tokens=max_new_tokens,
                           conf_mode=conf_mode, tau=tau, lam=lam, maxprob_thr=maxprob_thr,
                           mask_token_id=mcfg.mask_token_id, block_commit=block_commit, temperature=temperature,
                           sample_seed=sample_seed, seq_index=seq_index)
