"""fp64 CPU oracle of Dual-Stream Masking (Section 4.2): construction of the two-stream input and
the attention that its mask defines.

TEST INFRASTRUCTURE ONLY (same rules as wedlm_oracle.py: imported by the tests and by the benchmark's
CPU leg, shares nothing with the CUDA path and never calls it).

The physical input is the memory stream (the clean sequence, logical order) followed by the prediction
stream (the same sequence cut into blocks of B tokens, each block masked at its own ratio and reordered
observed-first with logical positions kept).  Both streams carry the position ids 0..L-1 (Eq. 8-9).
Which keys a row may look at is written here row by row over the 2L physical rows, straight from the
two rules of the paper's "Attention Pattern" paragraph (visible_columns; visibility stacks the rows into
one boolean matrix); attention is then plain softmax attention over each row's visible set.  Nothing is
tiled, blocked or reformulated as windows on a cache.

Readings of points the paper leaves open:
  * the memory stream attends causally to itself (it is the clean autoregressive context; the paper
    only states what prediction rows see);
  * "precede" inside a block includes the row itself (the diagonal), as in the decoding path;
  * a prediction row of block k sees memory rows at positions < k*B only: not the clean copy of its own
    block, in particular not its own clean token;
  * positions are 0-based.
Parity unpinned (nothing printed in the paper can confirm them): the first three readings above.  The
functions themselves are pinned against the rules as stated, by brute force and library special cases.
"""
from __future__ import annotations

from typing import Dict, Optional, Sequence

import numpy as np

from .wedlm_oracle import rope, to_f64


def construct(tokens: Sequence[int], masked: Sequence[int], block: int, mask_token_id: int) -> Dict[str, np.ndarray]:
    """Eq. 8-9 plus block-wise masking and intra-block reordering for one sequence of length L.

    masked[j] != 0 marks logical position j of the prediction stream as masked.  Returns, over the 2L
    physical rows (memory stream first): x_input, p_input, and for the prediction stream perm [L]
    (physical row L + i holds logical position perm[i]) and is_mask [L] (physical order)."""
    tok = np.asarray(tokens, dtype=np.int64)
    msk = np.asarray(masked).astype(bool)
    L = tok.shape[0]
    perm = np.zeros(L, np.int64)
    for start in range(0, L, block):
        idx = np.arange(start, min(start + block, L))
        obs = [j for j in idx if not msk[j]]
        mks = [j for j in idx if msk[j]]
        perm[start:start + len(idx)] = obs + mks            # observed to the front, masked to the back, order kept
    x_t = np.where(msk[perm], mask_token_id, tok[perm])
    x_input = np.concatenate([tok, x_t])
    p_input = np.concatenate([np.arange(L), perm])
    return dict(x_input=x_input, p_input=p_input, perm=perm, is_mask=msk[perm])


def visible_columns(a: int, L: int, block: int) -> np.ndarray:
    """Physical rows that physical row a may look at (ascending).  Rows 0..L-1 are the memory stream,
    rows L..2L-1 the prediction stream (block k = physical rows L + k*B .. L + (k+1)*B - 1)."""
    if a < L:
        return np.arange(0, a + 1)                           # memory stream: causal
    k = (a - L) // block
    memory = np.arange(0, min(k * block, L))                 # memory tokens whose positions precede block k
    own = np.arange(L + k * block, a + 1)                    # own block, physically not later than the row
    return np.concatenate([memory, own])


def visibility(L: int, block: int) -> np.ndarray:
    """vis[a, c] over the 2L physical rows."""
    vis = np.zeros((2 * L, 2 * L), dtype=bool)
    for a in range(2 * L):
        vis[a, visible_columns(a, L, block)] = True
    return vis


def attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, p_input: np.ndarray, block: int, *, theta: float,
              rope_style: int = 0, scale: Optional[float] = None, rows: Optional[Sequence[int]] = None) -> np.ndarray:
    """q [2L, Hq, D], k, v [2L, Hkv, D] in physical order -> out [2L, Hq, D] (float64): RoPE at p_input,
    then for every row softmax attention over visible_columns(row); query head h reads KV head
    h // (Hq // Hkv).  `rows` restricts the computed rows (the rest stay zero)."""
    qf, kf, vf = to_f64(q), to_f64(k), to_f64(v)
    N, Hq, D = qf.shape
    L = N // 2
    Hkv = kf.shape[1]
    G = Hq // Hkv
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    pos = np.asarray(p_input)
    k_rot = rope(kf, pos[:, None], theta, rope_style)
    out = np.zeros((N, Hq, D))
    for a in (range(N) if rows is None else rows):
        cols = visible_columns(a, L, block)
        q_rot = rope(qf[a], pos[a], theta, rope_style)
        for h in range(Hq):
            g = h // G
            s = scale * (k_rot[cols, g] @ q_rot[h])
            p = np.exp(s - s.max())
            p /= p.sum()
            out[a, h] = p @ vf[cols, g]
    return out


def attention_dense(q: np.ndarray, k: np.ndarray, v: np.ndarray, p_input: np.ndarray, block: int, *, theta: float,
                    rope_style: int = 0, scale: Optional[float] = None) -> np.ndarray:
    """The same quantity as `attention`, for all 2L rows at once: per head one dense score matrix over all
    2L x 2L (row, key) pairs, the pairs outside `visibility(L, block)` set to -inf, a row-wise softmax and one
    product with V.  It is the definition with the mask written as a matrix instead of as a list of columns
    per row; used where every row of a long sequence is compared (the row-by-row form takes minutes there)."""
    qf, kf, vf = to_f64(q), to_f64(k), to_f64(v)
    N, Hq, D = qf.shape
    L = N // 2
    G = Hq // kf.shape[1]
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    pos = np.asarray(p_input)
    q_rot = rope(qf, pos[:, None], theta, rope_style)
    k_rot = rope(kf, pos[:, None], theta, rope_style)
    vis = visibility(L, block)
    out = np.zeros((N, Hq, D))
    for h in range(Hq):
        g = h // G
        s = scale * (q_rot[:, h] @ k_rot[:, g].T)
        s[~vis] = -np.inf
        s -= s.max(axis=1, keepdims=True)
        np.exp(s, out=s)
        s /= s.sum(axis=1, keepdims=True)
        out[:, h] = s @ vf[:, g]
    return out
