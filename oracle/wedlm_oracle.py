"""fp64 CPU oracle for one WeDLM streaming-parallel-decoding step.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the hot path
computes.  It is imported by the tests, by the smoke check and by the benchmark's CPU-baseline
leg, and by nothing else; it shares no code with the CUDA library and never calls it.

Every real-valued quantity is computed in float64.  bf16 inputs arrive as uint16 bit patterns
and fp32 inputs as float32; both are widened exactly and never rounded again inside.

What follows the paper, by function:
  reorder                  Topological Reordering, Eq. 5-6, and the commit length of Algorithm 1
                           (line "n <- min{i : W[i] = [M]}"), read in logical order.
  rope                     RoPE indexed by supplied logical positions (Section 2.2, Eq. 2).
  window_attention         "a causal forward over the current window conditioned on the cached
                           prefix" (Section 5.2): plain softmax attention, written out.
  confidence               entropy H_i of the predicted distribution (Section 5.2), plus max-prob.
  sample_token             Sample(l_i) of Algorithm 1 at a temperature (Section 6.1 evaluates at
                           0.1): one draw from softmax(l / T), realised as arg-max of l / T plus
                           Gumbel noise from a counter-based generator keyed by (seed, sequence,
                           position, token).
  select_commit_refill     Algorithm 1, Commit / Predict / Refill, with Eq. 11 as selection score.
  step, decode_loop        the steps above in the order of Algorithm 1.

Readings of points the paper leaves open (all switchable by arguments):
  * commit length is the leading run of filled slots in LOGICAL order;
  * causal attention includes the diagonal (physical j <= i), as stock causal kernels do;
  * selection is non-strict (H~ <= tau, p_max >= thr);
  * if no mask passes, exactly one mask is filled: the one with the best score, leftmost on ties;
  * d_i is the logical slot distance to the leftmost mask after the commit;
  * entropy uses natural log on raw logits (also when sampling: the temperature shapes the
    draw, not the confidence); Sample() is greedy arg-max, lowest index on ties, unless a
    temperature > 0 is given;
  * RoPE pairs (d, d + D/2) ("rotate-half"); style 1 pairs (2d, 2d+1);
  * GQA: query head h reads KV head h // (Hq // Hkv);
  * positions are 0-based: slot j of a window on a prefix of length P has position id P + j.
Parity unpinned (readings that nothing printed in the paper can confirm): diagonal inclusion,
strictness of the threshold, the fallback rule, the max-prob mode, the RoPE pairing, the budget
rule for termination.  They are internally consistent and isolated behind arguments.
"""
from __future__ import annotations

from typing import Callable, Dict, List, Optional, Sequence, Tuple

import numpy as np


# ----------------------------------------------------------------------------------------
# input widening
# ----------------------------------------------------------------------------------------
def to_f64(x: np.ndarray) -> np.ndarray:
    """Widen a stored tensor exactly: uint16 = bf16 bit pattern, float32, or float64."""
    x = np.asarray(x)
    if x.dtype == np.uint16:
        return (x.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    return x.astype(np.float64)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float64 values to the nearest bf16 (ties to even); returned as float64.

    Only used to state what a bf16 cache should hold after staging (never inside attention)."""
    x = np.asarray(x, dtype=np.float64)
    m, e = np.frexp(x)                      # x = m * 2**e, 0.5 <= |m| < 1
    q = np.rint(m * 256.0) / 256.0          # 8 significant bits; rint is ties-to-even
    return np.ldexp(q, e)


# ----------------------------------------------------------------------------------------
# Topological Reordering (Eq. 5-6) and the commit length (Algorithm 1, Commit)
# ----------------------------------------------------------------------------------------
def reorder(filled: np.ndarray, prefix_len: np.ndarray,
            window_len: Optional[np.ndarray] = None, block_commit: bool = False) -> Dict[str, np.ndarray]:
    """Stable partition of each window: filled slots (ascending logical index) first, then masks
    (ascending).  pos_ids keeps each slot's logical position P + j.  Slots at or beyond
    window_len (a window that shrank at the end of generation) are treated as trailing masks.

    Returns perm, inv_perm, pos_ids [B,W] (indexed by physical slot), n_filled, n_commit [B]."""
    filled = np.asarray(filled)
    B, W = filled.shape
    perm = np.zeros((B, W), np.int32)
    inv = np.zeros((B, W), np.int32)
    pos = np.zeros((B, W), np.int32)
    n_filled = np.zeros(B, np.int32)
    n_commit = np.zeros(B, np.int32)
    for b in range(B):
        L = W if window_len is None else int(window_len[b])
        f = [bool(filled[b, j]) and j < L for j in range(W)]
        observed = [j for j in range(W) if f[j]]
        masked = [j for j in range(W) if not f[j]]
        order = observed + masked
        for i, j in enumerate(order):
            perm[b, i] = j
            inv[b, j] = i
            pos[b, i] = int(prefix_len[b]) + j
        n_filled[b] = len(observed)
        if block_commit:
            # block-wise baseline (Section 5.2, Fig. 2): nothing is committed until the whole block is final
            n_commit[b] = L if (len(observed) == L and L > 0) else 0
        else:
            n_commit[b] = masked[0] if masked else W
    return dict(perm=perm, inv_perm=inv, pos_ids=pos, n_filled=n_filled, n_commit=n_commit)


# ----------------------------------------------------------------------------------------
# RoPE at supplied logical positions
# ----------------------------------------------------------------------------------------
def rope(x: np.ndarray, pos: np.ndarray, theta: float, style: int = 0) -> np.ndarray:
    """Rotate the last axis of x (length D) by angles pos * theta**(-2d/D), d = 0..D/2-1.

    `pos` broadcasts against x.shape[:-1].  style 0 pairs (d, d+D/2); style 1 pairs (2d, 2d+1)."""
    x = np.asarray(x, dtype=np.float64)
    D = x.shape[-1]
    half = D // 2
    d = np.arange(half, dtype=np.float64)
    inv_freq = np.power(float(theta), -2.0 * d / D)
    ang = np.asarray(pos, dtype=np.float64)[..., None] * inv_freq
    c, s = np.cos(ang), np.sin(ang)
    out = np.empty_like(x)
    if style == 0:
        a, b = x[..., :half], x[..., half:]
        out[..., :half] = a * c - b * s
        out[..., half:] = b * c + a * s
    else:
        a, b = x[..., 0::2], x[..., 1::2]
        out[..., 0::2] = a * c - b * s
        out[..., 1::2] = b * c + a * s
    return out


# ----------------------------------------------------------------------------------------
# paged cache access and staging slots (Algorithm 1, "Extend (K, V)")
# ----------------------------------------------------------------------------------------
def gather_prefix(cache: np.ndarray, block_table_row: np.ndarray, n_tokens: int, g: int) -> np.ndarray:
    """Rows 0..n_tokens-1 of KV head g of one sequence, read through its block table -> [n, D]."""
    page = cache.shape[2]
    n_pages = (n_tokens + page - 1) // page
    if n_pages == 0:
        return np.zeros((0, cache.shape[3]), np.float64)
    rows = to_f64(cache[np.asarray(block_table_row[:n_pages], dtype=np.int64), g])
    return rows.reshape(n_pages * page, -1)[:n_tokens]


def stage_slots(block_table: np.ndarray, prefix_len: np.ndarray, W: int, page: int) -> np.ndarray:
    """Cache slot of physical window row i: table[(P+i)//page] * page + (P+i) % page."""
    B = block_table.shape[0]
    slots = np.zeros((B, W), np.int32)
    for b in range(B):
        for i in range(W):
            t = int(prefix_len[b]) + i
            slots[b, i] = int(block_table[b, t // page]) * page + t % page
    return slots


# ----------------------------------------------------------------------------------------
# window attention over the committed prefix + the physical causal window
# ----------------------------------------------------------------------------------------
def _softmax_rows(s: np.ndarray) -> np.ndarray:
    m = np.max(s, axis=-1, keepdims=True)
    e = np.exp(s - m)
    return e / np.sum(e, axis=-1, keepdims=True)


def window_attention(q, k, v, k_cache, v_cache, block_table, prefix_len, pos_ids, *,
                     theta: float, rope_style: int = 0, scale: Optional[float] = None,
                     include_diagonal: bool = True,
                     seqs: Optional[Sequence[int]] = None) -> Dict[str, np.ndarray]:
    """out[b,i,h] = sum_t softmax_t(scale * <q~[b,i,h], key_t>) value_t over
         t in {cached positions 0..P_b-1}  U  {window rows j <= i (physical order)},
    with q~, k~ rotated at the logical position ids and cached K already rotated at its own
    position.  q [B,W,Hq,D], k,v [B,W,Hkv,D] are in physical order.

    Returns out [B,W,Hq,D], q_rot, k_rot (float64).  `seqs` restricts the work to some b."""
    qf, kf, vf = to_f64(q), to_f64(k), to_f64(v)
    B, W, Hq, D = qf.shape
    Hkv = kf.shape[2]
    G = Hq // Hkv
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    pos = np.asarray(pos_ids)
    q_rot = rope(qf, pos[:, :, None], theta, rope_style)
    k_rot = rope(kf, pos[:, :, None], theta, rope_style)
    out = np.zeros((B, W, Hq, D), np.float64)
    # window row i may look at window row j iff j <= i (j < i without the diagonal)
    jj, ii = np.meshgrid(np.arange(W), np.arange(W))
    win_vis = (jj <= ii) if include_diagonal else (jj < ii)
    for b in (range(B) if seqs is None else seqs):
        P = int(prefix_len[b])
        for g in range(Hkv):
            keys = np.concatenate([gather_prefix(k_cache, block_table[b], P, g), k_rot[b, :, g]], 0)
            vals = np.concatenate([gather_prefix(v_cache, block_table[b], P, g), vf[b, :, g]], 0)
            vis = np.concatenate([np.ones((W, P), bool), win_vis], axis=1)      # [W, P+W]
            for h in range(g * G, (g + 1) * G):
                s = scale * (q_rot[b, :, h] @ keys.T)                           # [W, P+W]
                sees = vis.any(axis=1)                   # a row with no visible key outputs zeros
                s = np.where(vis, s, -np.inf)
                s[~sees] = 0.0
                p = _softmax_rows(s)
                p[~sees] = 0.0
                out[b, :, h] = p @ vals
    return dict(out=out, q_rot=q_rot, k_rot=k_rot)


def window_attention_row(q, k, v, k_cache, v_cache, block_table, prefix_len, pos_ids,
                         b: int, i: int, h: int, *, theta: float, rope_style: int = 0,
                         scale: Optional[float] = None) -> np.ndarray:
    """One output vector out[b,i,h,:] of window_attention (diagonal included), computed alone:
    used to sample full-size workloads."""
    W, Hq, D = q.shape[1], q.shape[2], q.shape[3]
    Hkv = k.shape[2]
    g = h // (Hq // Hkv)
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    P = int(prefix_len[b])
    pos = np.asarray(pos_ids[b])
    qv = rope(to_f64(q[b, i, h]), pos[i], theta, rope_style)
    kw = rope(to_f64(k[b, : i + 1, g]), pos[: i + 1], theta, rope_style)
    keys = np.concatenate([gather_prefix(k_cache, block_table[b], P, g), kw], 0)
    vals = np.concatenate([gather_prefix(v_cache, block_table[b], P, g), to_f64(v[b, : i + 1, g])], 0)
    s = scale * (keys @ qv)
    p = np.exp(s - s.max())
    p /= p.sum()
    return p @ vals


# ----------------------------------------------------------------------------------------
# per-row confidence over the vocabulary
# ----------------------------------------------------------------------------------------
def confidence(logits_rows: np.ndarray) -> Dict[str, np.ndarray]:
    """For each row x of logits [R, V]: arg-max (lowest index on ties), lse = ln sum exp x,
    p = exp(x - lse), max-prob = p[argmax], entropy H = -sum p ln p in nats (p = 0 adds 0)."""
    x = to_f64(logits_rows)
    if x.ndim == 1:
        x = x[None]
    R = x.shape[0]
    amax = np.zeros(R, np.int32)
    lse = np.zeros(R)
    maxprob = np.zeros(R)
    ent = np.zeros(R)
    for r in range(R):
        row = x[r]
        a = int(np.argmax(row))                # numpy returns the first occurrence
        m = row[a]
        lse[r] = m + np.log(np.sum(np.exp(row - m)))
        logp = row - lse[r]
        p = np.exp(logp)
        terms = np.where(p > 0.0, p * logp, 0.0)
        ent[r] = -np.sum(terms)
        maxprob[r] = p[a]
        amax[r] = a
    return dict(argmax=amax, lse=lse, maxprob=maxprob, entropy=ent)


# ----------------------------------------------------------------------------------------
# Sample(l_i) of Algorithm 1 at temperature T
# ----------------------------------------------------------------------------------------
# A draw from softmax(l / T) is the arg-max over v of l_v / T + g_v with g_v independent standard
# Gumbel variables (the Gumbel-max identity), g = -ln(-ln u), u uniform on (0, 1).  The uniforms
# come from a stateless generator so that a row's draw depends only on (seed, sequence index,
# logical position, token id) and not on how the work is cut up: u = ((h >> 9) + 1/2) / 2^23 with h
# a 32-bit integer hash (23 bits, so that u is also exact in single precision).  The hash is a xor-shift / odd-multiply finaliser; any implementation has
# to reproduce these integer steps exactly to draw the same tokens.
_M1 = np.uint32(0x7FEB352D)
_M2 = np.uint32(0x846CA68B)
_GOLD = np.uint32(0x9E3779B9)
_POSMUL = np.uint32(0x85EBCA6B)


def mix32(x) -> np.ndarray:
    """Bijective 32-bit finaliser: x ^= x>>16; x *= M1; x ^= x>>15; x *= M2; x ^= x>>16 (mod 2^32)."""
    x = np.asarray(x, dtype=np.uint32).copy()
    with np.errstate(over="ignore"):
        x ^= x >> np.uint32(16)
        x *= _M1
        x ^= x >> np.uint32(15)
        x *= _M2
        x ^= x >> np.uint32(16)
    return x


def sample_key(seed_lo: int, seed_hi: int, b: int, pos: int) -> np.uint32:
    """Row key: k1 = mix32(seed_lo + GOLD * b); key = mix32(k1 ^ seed_hi ^ (POSMUL * pos))."""
    with np.errstate(over="ignore"):
        k1 = mix32(np.uint32(seed_lo & 0xFFFFFFFF) + _GOLD * np.uint32(b & 0xFFFFFFFF))
        return mix32(k1 ^ np.uint32(seed_hi & 0xFFFFFFFF) ^ (_POSMUL * np.uint32(pos & 0xFFFFFFFF)))[()]


def sample_uniforms(key, V: int) -> np.ndarray:
    """u_v in (0, 1) for token ids 0..V-1: 23 high bits of mix32(key ^ GOLD * v), centred."""
    with np.errstate(over="ignore"):
        h = mix32(np.uint32(key) ^ (_GOLD * np.arange(V, dtype=np.uint32)))
    return ((h >> np.uint32(9)).astype(np.float64) + 0.5) * 2.0 ** -23


def sample_token(logits_row: np.ndarray, temperature: float, seed: Tuple[int, int], b: int, pos: int) -> Tuple[int, float]:
    """(token, margin): token = arg-max_v of l_v / T + g_v (lowest v on ties); margin = best minus
    second-best perturbed score (how far the draw is from flipping under rounding)."""
    x = to_f64(np.asarray(logits_row)).reshape(-1)
    u = sample_uniforms(sample_key(seed[0], seed[1], b, pos), x.shape[0])
    z = x / float(temperature) - np.log(-np.log(u))
    a = int(np.argmax(z))
    if z.shape[0] > 1:
        rest = np.delete(z, a)
        margin = float(z[a] - np.max(rest))
    else:
        margin = float("inf")
    return a, margin


# ----------------------------------------------------------------------------------------
# Commit / Predict / Refill of Algorithm 1 for one sequence
# ----------------------------------------------------------------------------------------
def select_commit_refill(tokens: Sequence[int], filled: Sequence[int], window_len: int,
                         prefix_len: int, mask_argmax: Sequence[int],
                         mask_entropy: Sequence[float], mask_maxprob: Sequence[float], *,
                         conf_mode: str, tau: float, lam: float, maxprob_thr: float,
                         mask_token_id: int, remaining_budget: Optional[int] = None,
                         fallback: bool = True, block_commit: bool = False) -> Dict[str, object]:
    """tokens/filled: the window in LOGICAL order (W slots, the first window_len active).
    mask_*[k] are the statistics of the k-th active mask in ascending logical order (that is the
    physical row n_filled + k after reordering).

    Order of operations is Algorithm 1's: commit the leading filled run (n slots), drop them,
    select among the remaining masks by Eq. 11 (d counted from the leftmost mask), fill the
    selected with their arg-max, append min(n, budget) fresh masks."""
    W = len(tokens)
    L = int(window_len)
    tok = [int(t) for t in tokens]
    fil = [1 if (filled[j] and j < L) else 0 for j in range(W)]
    # Commit: leftmost contiguous filled prefix.
    n = 0
    while n < L and fil[n]:
        n += 1
    if block_commit and n < L:
        n = 0                           # block-wise baseline: all active slots or nothing
    committed = tok[:n]
    # Masks of the current window, ascending; k-th one owns statistics row k.
    masks = [j for j in range(L) if not fil[j]]
    score: List[float] = []
    chosen: List[int] = []
    if masks:
        j0 = masks[0]
        for kk, j in enumerate(masks):
            if conf_mode == "entropy":
                sc = float(mask_entropy[kk]) + lam * (j - j0)        # Eq. 11
                ok = sc <= tau
            else:
                sc = -float(mask_maxprob[kk])                        # lower is better
                ok = float(mask_maxprob[kk]) >= maxprob_thr
            score.append(sc)
            if ok:
                chosen.append(kk)
        if not chosen and fallback:
            best = min(range(len(masks)), key=lambda kk: (score[kk], kk))
            chosen = [best]
    for kk in chosen:
        tok[masks[kk]] = int(mask_argmax[kk])
        fil[masks[kk]] = 1
    # Drop the committed slots, refill with fresh masks (limited by the remaining budget).
    r = n if remaining_budget is None else min(n, int(remaining_budget))
    new_len = L - n + r
    new_tok = tok[n:L] + [mask_token_id] * r
    new_fil = fil[n:L] + [0] * r
    pad = W - new_len
    new_tok += [mask_token_id] * pad
    new_fil += [0] * pad
    return dict(committed_tokens=committed, committed_count=n,
                filled_slots=[masks[kk] for kk in chosen], filled_count=len(chosen),
                window_tokens=new_tok, filled=new_fil, window_len=new_len,
                prefix_len=int(prefix_len) + n,
                remaining_budget=None if remaining_budget is None else int(remaining_budget) - r,
                mask_slots=masks, scores=score)


# ----------------------------------------------------------------------------------------
# one full step, batched (reorder -> attention -> confidence -> commit/predict/refill)
# ----------------------------------------------------------------------------------------
def step(inp: Dict[str, np.ndarray], *, theta: float, rope_style: int = 0, conf_mode: str,
         tau: float, lam: float, maxprob_thr: float, mask_token_id: int, page_size: int,
         window_len: Optional[np.ndarray] = None, remaining_budget: Optional[np.ndarray] = None,
         with_attention: bool = True, block_commit: bool = False, temperature: float = 0.0,
         sample_seed: Tuple[int, int] = (0, 0)) -> Dict[str, object]:
    """All outputs of one decoding step for the arrays of workloads.make_step().  With
    temperature > 0 the token of every mask row is sampled: "sampled" [B,W] holds the draw of each
    mask row (-1 elsewhere), "sample_margin" its gap to the runner-up, and the selected slots are
    filled with the draws; "argmax" stays the greedy arg-max."""
    filled, prefix_len = inp["filled"], inp["prefix_len"]
    B, W = filled.shape
    ro = reorder(filled, prefix_len, window_len, block_commit)
    res: Dict[str, object] = dict(ro)
    res["tokens_phys"] = np.take_along_axis(np.asarray(inp["window_tokens"]), ro["perm"], axis=1)
    res["kv_slot_idx"] = stage_slots(inp["block_table"], prefix_len, W, page_size)
    if with_attention:
        res.update(window_attention(inp["q"], inp["k"], inp["v"], inp["k_cache"], inp["v_cache"],
                                    inp["block_table"], prefix_len, ro["pos_ids"],
                                    theta=theta, rope_style=rope_style))
    argmax = np.full((B, W), -1, np.int32)
    ent = np.full((B, W), np.nan)
    mp = np.full((B, W), np.nan)
    lse = np.full((B, W), np.nan)
    margin = np.full((B, W), np.inf)
    sampled = np.full((B, W), -1, np.int32)
    per_seq = []
    for b in range(B):
        L = W if window_len is None else int(window_len[b])
        nf = int(ro["n_filled"][b])
        n_mask = L - nf
        if n_mask > 0:
            c = confidence(inp["logits"][b, nf:nf + n_mask])
            argmax[b, nf:nf + n_mask] = c["argmax"]
            ent[b, nf:nf + n_mask] = c["entropy"]
            mp[b, nf:nf + n_mask] = c["maxprob"]
            lse[b, nf:nf + n_mask] = c["lse"]
            if temperature > 0.0:
                for i in range(nf, nf + n_mask):
                    sampled[b, i], margin[b, i] = sample_token(inp["logits"][b, i], temperature, sample_seed, b,
                                                               int(ro["pos_ids"][b, i]))
        fill_with = sampled if temperature > 0.0 else argmax
        per_seq.append(select_commit_refill(
            inp["window_tokens"][b], filled[b], L, int(prefix_len[b]),
            fill_with[b, nf:nf + n_mask], ent[b, nf:nf + n_mask], mp[b, nf:nf + n_mask],
            conf_mode=conf_mode, tau=tau, lam=lam, maxprob_thr=maxprob_thr,
            mask_token_id=mask_token_id,
            remaining_budget=None if remaining_budget is None else int(remaining_budget[b]),
            block_commit=block_commit))
    res.update(argmax=argmax, entropy=ent, maxprob=mp, lse=lse, per_seq=per_seq, sampled=sampled,
               sample_margin=margin)
    return res


# ----------------------------------------------------------------------------------------
# Algorithm 1 as a loop over a caller-supplied model
# ----------------------------------------------------------------------------------------
def decode_loop(forward: Callable[[List[int], List[int], List[int]], np.ndarray], *,
                prefix_len: int, window: int, max_new_tokens: int, conf_mode: str, tau: float,
                lam: float, maxprob_thr: float, mask_token_id: int,
                max_steps: int = 100000, block_commit: bool = False, temperature: float = 0.0,
                sample_seed: Tuple[int, int] = (0, 0), seq_index: int = 0) -> Dict[str, object]:
    """Streaming Parallel Decoding (Algorithm 1) for one sequence.

    forward(y, tokens_phys, pos_ids) -> logits [W_len, V]: the causal forward of the reordered
    window on top of the committed text y; row i predicts physical slot i.  The window starts as
    min(W, budget) masks; every slot created counts against max_new_tokens."""
    W = window
    L = min(W, max_new_tokens)
    budget = max_new_tokens - L
    tok = [mask_token_id] * W
    fil = [0] * W
    y: List[int] = []
    P = prefix_len
    n_fwd = 0
    trace = []
    steps = 0
    while L > 0 and steps < max_steps:
        ro = reorder(np.asarray([fil], np.uint8), np.asarray([P]), np.asarray([L]))
        perm = ro["perm"][0][:L]
        nf = int(ro["n_filled"][0])
        logits = np.asarray(forward(list(y), [tok[j] for j in perm], [int(p) for p in ro["pos_ids"][0][:L]]))
        n_fwd += L
        c = confidence(logits[nf:L]) if L > nf else dict(argmax=[], entropy=[], maxprob=[])
        if temperature > 0.0 and L > nf:
            c["argmax"] = [sample_token(logits[i], temperature, sample_seed, seq_index, int(ro["pos_ids"][0][i]))[0]
                           for i in range(nf, L)]
        r = select_commit_refill(tok, fil, L, P, c["argmax"], c["entropy"], c["maxprob"],
                                 conf_mode=conf_mode, tau=tau, lam=lam, maxprob_thr=maxprob_thr,
                                 mask_token_id=mask_token_id, remaining_budget=budget, block_commit=block_commit)
        y += r["committed_tokens"]
        trace.append(dict(window_len=L, committed=r["committed_count"], filled=r["filled_count"],
                          pos_ids=[int(p) for p in ro["pos_ids"][0][:L]]))
        tok, fil, L, P, budget = r["window_tokens"], r["filled"], r["window_len"], r["prefix_len"], r["remaining_budget"]
        steps += 1
    return dict(y=y, steps=steps, n_fwd=n_fwd, p_cache=(len(y) / n_fwd if n_fwd else 0.0), trace=trace)
