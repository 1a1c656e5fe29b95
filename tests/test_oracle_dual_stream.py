"""Pins for the Dual-Stream Masking oracle (Section 4.2, Eq. 8-9 and the "Attention Pattern" rules).

The construction is pinned by an example worked by hand from the paper's description; the mask by a
scalar predicate written independently from the two rules, by counting, and by the textbook special case
(the memory stream is a lower-triangular causal mask); the attention by library routines on the special
cases that reduce to them (causal attention for the memory stream, unmasked attention over the visible
set for the last row of a block), by the clean-copy invariant (an unmasked, unpermuted prediction stream
that repeats the memory stream must reproduce causal attention row for row, which fails if the streams
did not share one position frame), and by leak tests (perturbing an invisible key changes nothing)."""
import numpy as np
import torch

from oracle import dual_stream_oracle as ds
from oracle import wedlm_oracle as orc


def test_construction_worked_example():
    # L = 7, B = 3: blocks {0,1,2}, {3,4,5}, {6}.  Masked logical positions: 0, 2 | 4 | none.
    tokens = [10, 11, 12, 13, 14, 15, 16]
    masked = [1, 0, 1, 0, 1, 0, 0]
    r = ds.construct(tokens, masked, block=3, mask_token_id=99)
    # memory stream untouched; prediction stream per block: observed first (order kept), then masked
    assert r["x_input"].tolist() == [10, 11, 12, 13, 14, 15, 16] + [11, 99, 99] + [13, 15, 99] + [16]
    assert r["p_input"].tolist() == [0, 1, 2, 3, 4, 5, 6] + [1, 0, 2] + [3, 5, 4] + [6]
    assert r["is_mask"].tolist() == [False, True, True, False, False, True, False]
    # every block keeps its own positions: reordering never crosses a block boundary
    for start in (0, 3, 6):
        blk = r["perm"][start:start + 3]
        assert sorted(blk.tolist()) == list(range(start, min(start + 3, 7)))


def test_construction_nothing_masked_and_everything_masked():
    tokens = list(range(100, 110))
    r = ds.construct(tokens, [0] * 10, block=4, mask_token_id=7)
    assert r["x_input"].tolist() == tokens + tokens and r["p_input"].tolist() == list(range(10)) * 2
    r = ds.construct(tokens, [1] * 10, block=4, mask_token_id=7)
    assert r["x_input"].tolist() == tokens + [7] * 10 and r["p_input"].tolist() == list(range(10)) * 2


def _may_see(a, c, L, B):
    """The two rules, as a scalar predicate written apart from the oracle."""
    if a < L:                      # memory row
        return c <= a
    ka = (a - L) // B
    if c < L:                      # memory key: logical position c must precede block ka
        return c < ka * B
    kc = (c - L) // B
    return kc == ka and c <= a     # prediction key: same block, not physically later


def test_visibility_matches_the_rules_by_brute_force():
    for L, B in ((7, 3), (12, 4), (9, 9), (5, 1), (10, 32)):
        vis = ds.visibility(L, B)
        want = np.array([[_may_see(a, c, L, B) for c in range(2 * L)] for a in range(2 * L)])
        assert np.array_equal(vis, want), (L, B)
        # textbook special case: the memory stream alone is the causal lower triangle
        assert np.array_equal(vis[:L, :L], np.tril(np.ones((L, L), bool)))
        assert not vis[:L, L:].any()                       # memory never looks at the prediction stream
        for i in range(L):                                 # counting: k*B memory keys + r + 1 own keys
            k, r = divmod(i, B)
            assert vis[L + i].sum() == min(k * B, L) + r + 1
            assert not vis[L + i, k * B:L].any()           # never the clean copy of its own or later blocks
            assert not vis[L + i, L:L + k * B].any()       # never earlier prediction blocks


def _rand(L, Hq, Hkv, D, seed):
    g = np.random.default_rng(seed)
    q = g.standard_normal((2 * L, Hq, D))
    k = g.standard_normal((2 * L, Hkv, D))
    v = g.standard_normal((2 * L, Hkv, D))
    return q, k, v


def _sdpa(q, k, v, causal):
    """[n, H, D] arrays -> torch scaled_dot_product_attention in float64 (GQA by repeating KV heads)."""
    G = q.shape[1] // k.shape[1]
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]
    tk = torch.from_numpy(np.repeat(k, G, axis=1)).permute(1, 0, 2)[None]
    tv = torch.from_numpy(np.repeat(v, G, axis=1)).permute(1, 0, 2)[None]
    o = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=causal)
    return o[0].permute(1, 0, 2).numpy()


def test_memory_stream_is_library_causal_attention():
    L, B, Hq, Hkv, D, theta = 13, 4, 4, 2, 16, 1.0e4
    q, k, v = _rand(L, Hq, Hkv, D, 1)
    masked = np.random.default_rng(2).random(L) < 0.5
    c = ds.construct(np.arange(L), masked, B, 999)
    out = ds.attention(q, k, v, c["p_input"], B, theta=theta)
    pos = np.arange(L)
    want = _sdpa(orc.rope(q[:L], pos[:, None], theta), orc.rope(k[:L], pos[:, None], theta), v[:L], causal=True)
    np.testing.assert_allclose(out[:L], want, rtol=1e-10, atol=1e-12)


def test_last_row_of_a_block_is_unmasked_attention_over_its_visible_set():
    L, B, Hq, Hkv, D, theta = 12, 4, 2, 1, 8, 1.0e4
    q, k, v = _rand(L, Hq, Hkv, D, 3)
    masked = np.array([0, 1, 0, 1, 1, 1, 0, 0, 0, 0, 0, 1])
    c = ds.construct(np.arange(L), masked, B, 999)
    out = ds.attention(q, k, v, c["p_input"], B, theta=theta)
    p = c["p_input"]
    for kblk in range(3):
        a = L + kblk * B + B - 1
        cols = list(range(kblk * B)) + list(range(L + kblk * B, a + 1))
        want = _sdpa(orc.rope(q[a:a + 1], p[a:a + 1, None], theta), orc.rope(k[cols], p[cols][:, None], theta), v[cols],
                     causal=False)
        np.testing.assert_allclose(out[a], want[0], rtol=1e-10, atol=1e-12)


def test_clean_copy_prediction_stream_reproduces_causal_attention():
    # nothing masked, so no reordering: if the prediction stream repeats the memory stream's q, k, v, row L + i
    # sees memory[0, kB) and the copies of memory[kB, i]: the same keys, values and positions as memory row i
    L, B, Hq, Hkv, D, theta = 11, 4, 4, 2, 16, 1.0e6
    q, k, v = _rand(L, Hq, Hkv, D, 4)
    q[L:], k[L:], v[L:] = q[:L], k[:L], v[:L]
    c = ds.construct(np.arange(L), np.zeros(L, int), B, 999)
    out = ds.attention(q, k, v, c["p_input"], B, theta=theta)
    np.testing.assert_allclose(out[L:], out[:L], rtol=1e-10, atol=1e-12)


def test_invisible_keys_cannot_leak_and_visible_ones_matter():
    L, B, Hq, Hkv, D, theta = 12, 4, 2, 2, 8, 1.0e4
    q, k, v = _rand(L, Hq, Hkv, D, 5)
    masked = np.random.default_rng(6).random(L) < 0.6
    c = ds.construct(np.arange(L), masked, B, 999)
    base = ds.attention(q, k, v, c["p_input"], B, theta=theta)
    a = L + 1 * B + 1                                # block 1, second physical row
    for col, visible in ((2, True), (3, True), (4, False), (7, False), (L + 0, False), (L + 3, False), (L + 4, True),
                         (L + 5, True), (L + 6, False), (L + 8, False), (11, False)):
        k2, v2 = k.copy(), v.copy()
        k2[col] += 1.0
        v2[col] -= 2.0
        out = ds.attention(q, k2, v2, c["p_input"], B, theta=theta, rows=[a])
        changed = not np.allclose(out[a], base[a], rtol=0, atol=1e-9)
        assert changed == visible, (col, visible)


def test_shared_position_frame_and_shift_invariance():
    L, B, Hq, Hkv, D, theta = 10, 5, 2, 1, 8, 1.0e4
    q, k, v = _rand(L, Hq, Hkv, D, 7)
    masked = np.random.default_rng(8).random(L) < 0.5
    c = ds.construct(np.arange(L), masked, B, 999)
    base = ds.attention(q, k, v, c["p_input"], B, theta=theta)
    shifted = ds.attention(q, k, v, c["p_input"] + 37, B, theta=theta)
    np.testing.assert_allclose(shifted, base, rtol=1e-9, atol=1e-11)      # RoPE is relative
    # but moving only the prediction stream to another frame changes its rows (it reads memory keys)
    p2 = c["p_input"].copy()
    p2[L:] += L
    moved = ds.attention(q, k, v, p2, B, theta=theta)
    assert not np.allclose(moved[L + B:], base[L + B:], atol=1e-6)
    np.testing.assert_allclose(moved[:L], base[:L], rtol=1e-12)


def test_dense_form_equals_the_row_by_row_form():
    """attention_dense writes the mask as a matrix; attention lists each row's visible columns.  Same numbers."""
    rng = np.random.default_rng(41)
    for L, B, Hq, Hkv, D in ((13, 4, 4, 2, 8), (32, 8, 2, 1, 16), (7, 16, 3, 3, 4)):
        q = rng.standard_normal((2 * L, Hq, D))
        k = rng.standard_normal((2 * L, Hkv, D))
        v = rng.standard_normal((2 * L, Hkv, D))
        c = ds.construct(rng.integers(0, 50, size=L), rng.random(L) < 0.5, B, 99)
        a = ds.attention(q, k, v, c["p_input"], B, theta=1.0e4)
        b = ds.attention_dense(q, k, v, c["p_input"], B, theta=1.0e4)
        np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-13)
