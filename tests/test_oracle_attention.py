"""Pins for the oracle's RoPE and window attention.

Each test compares the oracle with something that is not the oracle: a brute-force loop written
from the visibility rule in words, a library routine (torch SDPA in float64), a closed form, or
an invariance the mathematics fixes."""
import cmath
import itertools
import math

import numpy as np
import pytest
import torch

from oracle import wedlm_oracle as orc


def _identity_cache(K, V, page=4):
    """Pack per-sequence [P, Hkv, D] prefixes into a paged cache with an identity block table."""
    B = len(K)
    Hkv, D = K[0].shape[1], K[0].shape[2]
    W_extra = 64
    pages = [(k.shape[0] + W_extra + page - 1) // page for k in K]
    maxp = max(pages)
    table = np.full((B, maxp), -1, np.int32)
    kc = np.zeros((sum(pages), Hkv, page, D))
    vc = np.zeros_like(kc)
    at = 0
    for b in range(B):
        table[b, :pages[b]] = np.arange(at, at + pages[b])
        for t in range(K[b].shape[0]):
            kc[at + t // page, :, t % page] = K[b][t]
            vc[at + t // page, :, t % page] = V[b][t]
        at += pages[b]
    return kc, vc, table


def _rot_pair(a, b, ang):
    z = complex(a, b) * cmath.exp(1j * ang)
    return z.real, z.imag


def _rope_brute(x, pos, theta, style):
    """RoPE through complex multiplication, one pair at a time."""
    D = len(x)
    out = [0.0] * D
    for d in range(D // 2):
        ang = pos * theta ** (-2.0 * d / D)
        i0, i1 = (d, d + D // 2) if style == 0 else (2 * d, 2 * d + 1)
        out[i0], out[i1] = _rot_pair(x[i0], x[i1], ang)
    return out


@pytest.mark.parametrize("style", [0, 1])
def test_rope_matches_complex_rotation(style):
    rng = np.random.default_rng(1)
    x = rng.standard_normal((3, 8))
    pos = np.array([0, 5, 1234])
    got = orc.rope(x, pos, 10000.0, style)
    for r in range(3):
        np.testing.assert_allclose(got[r], _rope_brute(x[r].tolist(), int(pos[r]), 10000.0, style), atol=1e-12)


def test_rope_d2_is_a_plane_rotation_by_pos_radians():
    # D = 2: a single pair with frequency theta^0 = 1, so the angle is the position itself.
    got = orc.rope(np.array([[1.0, 0.0]]), np.array([3]), 12345.0)
    np.testing.assert_allclose(got[0], [math.cos(3.0), math.sin(3.0)], atol=1e-14)
    # position 0 is the identity
    x = np.arange(16.0)
    np.testing.assert_array_equal(orc.rope(x[None], np.array([0]), 1e6)[0], x)


def _brute_logical_attention(ql, kl, vl, Kc, Vc, filled, P, theta, G, scale):
    """Attention computed in LOGICAL layout under the visibility the reordering implies:
    every slot sees the whole committed prefix; an observed slot sees observed slots at an
    earlier-or-equal logical index; a mask slot sees every observed slot and the mask slots at
    an earlier-or-equal logical index.  Pure Python loops."""
    W, Hq, D = len(ql), len(ql[0]), len(ql[0][0])
    out = [[[0.0] * D for _ in range(Hq)] for _ in range(W)]
    for a in range(W):
        for h in range(Hq):
            g = h // G
            qa = _rope_brute(ql[a][h], P + a, theta, 0)
            keys, vals = [], []
            for t in range(P):
                keys.append(Kc[t][g])
                vals.append(Vc[t][g])
            for b in range(W):
                if filled[b]:
                    vis = (not filled[a]) or b <= a
                else:
                    vis = (not filled[a]) and b <= a
                if vis:
                    keys.append(_rope_brute(kl[b][g], P + b, theta, 0))
                    vals.append(vl[b][g])
            s = [scale * sum(x * y for x, y in zip(qa, kk)) for kk in keys]
            m = max(s)
            e = [math.exp(x - m) for x in s]
            z = sum(e)
            for d in range(D):
                out[a][h][d] = sum(e[t] * vals[t][d] for t in range(len(keys))) / z
    return out


@pytest.mark.parametrize("W,P", [(4, 3), (5, 0), (6, 5)])
def test_reordered_causal_attention_equals_logical_attention_under_visibility_mask(W, P):
    """Section 4.1: after reordering, plain causal attention gives every mask the full observed
    context.  All 2^W fill patterns."""
    Hq, Hkv, D, theta = 2, 1, 4, 100.0
    G = Hq // Hkv
    rng = np.random.default_rng(W * 100 + P)
    ql, kl, vl = rng.standard_normal((W, Hq, D)), rng.standard_normal((W, Hkv, D)), rng.standard_normal((W, Hkv, D))
    Kc, Vc = rng.standard_normal((P, Hkv, D)), rng.standard_normal((P, Hkv, D))
    kc, vc, table = _identity_cache([Kc], [Vc])
    scale = 1.0 / math.sqrt(D)
    for f in itertools.product([0, 1], repeat=W):
        perm = sorted(range(W), key=lambda j: (0 if f[j] else 1, j))     # the test's own reordering
        pos = np.array([[P + j for j in perm]])
        got = orc.window_attention(ql[perm][None], kl[perm][None], vl[perm][None], kc, vc, table,
                                   np.array([P]), pos, theta=theta)["out"][0]
        want = _brute_logical_attention(ql.tolist(), kl.tolist(), vl.tolist(), Kc.tolist(), Vc.tolist(),
                                        f, P, theta, G, scale)
        for i, j in enumerate(perm):
            np.testing.assert_allclose(got[i], np.array(want[j]), atol=1e-12, rtol=0)


@pytest.mark.parametrize("Hq,Hkv", [(4, 2), (4, 4), (8, 1)])
def test_fully_observed_window_is_ordinary_causal_attention(Hq, Hkv):
    """All slots filled: identity permutation, consecutive positions; the result must equal a
    library causal attention (torch SDPA, float64) of W new tokens on top of the prefix."""
    B, W, P, D, theta = 2, 7, 19, 8, 10000.0
    G = Hq // Hkv
    rng = np.random.default_rng(5)
    q, k, v = rng.standard_normal((B, W, Hq, D)), rng.standard_normal((B, W, Hkv, D)), rng.standard_normal((B, W, Hkv, D))
    Ks = [rng.standard_normal((P, Hkv, D)) for _ in range(B)]
    Vs = [rng.standard_normal((P, Hkv, D)) for _ in range(B)]
    kc, vc, table = _identity_cache(Ks, Vs)
    ro = orc.reorder(np.ones((B, W), np.uint8), np.full(B, P))
    got = orc.window_attention(q, k, v, kc, vc, table, np.full(B, P), ro["pos_ids"], theta=theta)["out"]
    for b in range(B):
        # library path: rotate with the complex formulation, expand KV heads, call SDPA
        qr = np.array([[_rope_brute(q[b, i, h].tolist(), P + i, theta, 0) for h in range(Hq)] for i in range(W)])
        kr = np.array([[_rope_brute(k[b, i, g].tolist(), P + i, theta, 0) for g in range(Hkv)] for i in range(W)])
        keys = np.concatenate([Ks[b], kr], 0).repeat(G, axis=1)      # [P+W, Hq, D]
        vals = np.concatenate([Vs[b], v[b]], 0).repeat(G, axis=1)
        mask = torch.ones(W, P + W, dtype=torch.bool).tril(diagonal=P)
        ref = torch.nn.functional.scaled_dot_product_attention(
            torch.tensor(qr).permute(1, 0, 2)[None], torch.tensor(keys).permute(1, 0, 2)[None],
            torch.tensor(vals).permute(1, 0, 2)[None], attn_mask=mask)[0].permute(1, 0, 2).numpy()
        np.testing.assert_allclose(got[b], ref, atol=1e-12, rtol=0)


def test_position_shift_invariance():
    """RoPE scores depend on position differences only: shifting every position id by a constant,
    with the cached keys re-rotated consistently, leaves the outputs unchanged."""
    B, W, P, Hq, Hkv, D, theta = 1, 5, 9, 2, 1, 8, 500.0
    rng = np.random.default_rng(9)
    q, k, v = rng.standard_normal((B, W, Hq, D)), rng.standard_normal((B, W, Hkv, D)), rng.standard_normal((B, W, Hkv, D))
    K_raw, Vc = rng.standard_normal((P, Hkv, D)), rng.standard_normal((P, Hkv, D))
    f = np.array([[1, 0, 1, 0, 0]], np.uint8)
    outs = []
    for shift in (0, 17):
        Kc = np.array([[_rope_brute(K_raw[t, g].tolist(), t + shift, theta, 0) for g in range(Hkv)] for t in range(P)])
        kc, vc, table = _identity_cache([Kc], [Vc])
        ro = orc.reorder(f, np.array([P]))
        outs.append(orc.window_attention(q, k, v, kc, vc, table, np.array([P]), ro["pos_ids"] + shift, theta=theta)["out"])
    np.testing.assert_allclose(outs[0], outs[1], atol=1e-10, rtol=0)


def test_softmax_special_cases():
    B, W, Hq, Hkv, D = 1, 3, 2, 2, 4
    rng = np.random.default_rng(2)
    q, k = rng.standard_normal((B, W, Hq, D)), rng.standard_normal((B, W, Hkv, D))
    # every value row identical -> the output is that row whatever the scores are
    row = rng.standard_normal(D)
    v = np.broadcast_to(row, (B, W, Hkv, D)).copy()
    Kc = rng.standard_normal((6, Hkv, D))
    kc, vc, table = _identity_cache([Kc], [np.broadcast_to(row, (6, Hkv, D)).copy()])
    pos = np.array([[6, 7, 8]])
    got = orc.window_attention(q, k, v, kc, vc, table, np.array([6]), pos, theta=1e4)["out"]
    np.testing.assert_allclose(got, np.broadcast_to(row, got.shape), atol=1e-13)
    # empty prefix: physical row 0 sees a single key (itself) -> output = its own value
    v2 = rng.standard_normal((B, W, Hkv, D))
    got = orc.window_attention(q, k, v2, kc, vc, table, np.array([0]), np.array([[0, 1, 2]]), theta=1e4)["out"]
    np.testing.assert_allclose(got[0, 0], v2[0, 0], atol=1e-13)


def test_paging_invariance_and_slot_formula():
    """The same logical cache behind an identity block table and behind a scrambled one gives the
    same outputs; staging slots follow table[(P+i)//page]*page + (P+i)%page across page edges."""
    W, Hq, Hkv, D, page, theta = 6, 2, 1, 4, 4, 1e4
    rng = np.random.default_rng(3)
    for P in (0, 1, 3, 4, 7, 15, 16):
        Kc, Vc = rng.standard_normal((P, Hkv, D)), rng.standard_normal((P, Hkv, D))
        kc, vc, table = _identity_cache([Kc], [Vc], page=page)
        n_pages = kc.shape[0]
        shuffle = rng.permutation(n_pages)
        kc2, vc2 = np.zeros_like(kc), np.zeros_like(vc)
        kc2[shuffle] = kc
        vc2[shuffle] = vc
        table2 = np.where(table >= 0, shuffle[np.maximum(table, 0)], -1).astype(np.int32)
        q, k, v = rng.standard_normal((1, W, Hq, D)), rng.standard_normal((1, W, Hkv, D)), rng.standard_normal((1, W, Hkv, D))
        pos = np.array([[P + j for j in (0, 2, 3, 1, 4, 5)]])
        a = orc.window_attention(q, k, v, kc, vc, table, np.array([P]), pos, theta=theta)["out"]
        b = orc.window_attention(q, k, v, kc2, vc2, table2, np.array([P]), pos, theta=theta)["out"]
        np.testing.assert_array_equal(a, b)
        slots = orc.stage_slots(table2, np.array([P]), W, page)[0]
        for i in range(W):
            assert slots[i] == table2[0, (P + i) // page] * page + (P + i) % page
        # consecutive rows are consecutive inside a page and jump at page edges
        assert len(set(slots.tolist())) == W


def test_stage_slots_hand_worked_values():
    """Cache slots of the staged window rows, worked by hand (slot = physical page * page size + offset):
    pages of 4 tokens, block table [5, 2, 9].  A prefix of 7 puts row 0 at token 7 = last row of logical
    page 1 (physical page 2 -> slot 11) and rows 1..4 at tokens 8..11 = logical page 2 (physical page 9
    -> slots 36..39).  A prefix on a page edge (8) starts a fresh page; a prefix of 3 straddles pages 5 and 2."""
    table = np.array([[5, 2, 9]], np.int32)
    assert orc.stage_slots(table, np.array([7]), 5, 4)[0].tolist() == [11, 36, 37, 38, 39]
    assert orc.stage_slots(table, np.array([8]), 4, 4)[0].tolist() == [36, 37, 38, 39]
    assert orc.stage_slots(table, np.array([3]), 3, 4)[0].tolist() == [23, 8, 9]
    assert orc.stage_slots(table, np.array([0]), 2, 4)[0].tolist() == [20, 21]
    # two sequences, each through its own table row
    table2 = np.array([[1, 0], [0, 3]], np.int32)
    assert orc.stage_slots(table2, np.array([1, 3]), 2, 4).tolist() == [[5, 6], [3, 12]]


def test_gqa_equals_replicated_kv_heads():
    B, W, P, Hq, Hkv, D, theta = 1, 4, 5, 6, 2, 4, 1e4
    G = Hq // Hkv
    rng = np.random.default_rng(4)
    q, k, v = rng.standard_normal((B, W, Hq, D)), rng.standard_normal((B, W, Hkv, D)), rng.standard_normal((B, W, Hkv, D))
    Kc, Vc = rng.standard_normal((P, Hkv, D)), rng.standard_normal((P, Hkv, D))
    kc, vc, table = _identity_cache([Kc], [Vc])
    kcr, vcr, table_r = _identity_cache([Kc.repeat(G, axis=1)], [Vc.repeat(G, axis=1)])
    pos = np.array([[P + j for j in (1, 3, 0, 2)]])
    a = orc.window_attention(q, k, v, kc, vc, table, np.array([P]), pos, theta=theta)["out"]
    b = orc.window_attention(q, k.repeat(G, axis=2), v.repeat(G, axis=2), kcr, vcr, table_r,
                             np.array([P]), pos, theta=theta)["out"]
    np.testing.assert_allclose(a, b, atol=1e-14)


def test_single_row_routine_agrees_with_the_batched_one():
    B, W, P, Hq, Hkv, D, theta = 2, 5, 11, 4, 2, 8, 1e6
    rng = np.random.default_rng(6)
    q, k, v = rng.standard_normal((B, W, Hq, D)), rng.standard_normal((B, W, Hkv, D)), rng.standard_normal((B, W, Hkv, D))
    Ks = [rng.standard_normal((P, Hkv, D)) for _ in range(B)]
    Vs = [rng.standard_normal((P, Hkv, D)) for _ in range(B)]
    kc, vc, table = _identity_cache(Ks, Vs)
    ro = orc.reorder(np.array([[1, 0, 1, 1, 0], [0, 0, 1, 0, 1]], np.uint8), np.full(B, P))
    full = orc.window_attention(q, k, v, kc, vc, table, np.full(B, P), ro["pos_ids"], theta=theta)["out"]
    for (b, i, h) in [(0, 0, 0), (1, 4, 3), (0, 2, 1)]:
        one = orc.window_attention_row(q, k, v, kc, vc, table, np.full(B, P), ro["pos_ids"], b, i, h, theta=theta)
        np.testing.assert_allclose(one, full[b, i, h], atol=1e-13)


def test_bf16_widening_and_rounding():
    bits = np.array([0x3F80, 0xC020, 0x0000, 0x4049], np.uint16)   # 1.0, -2.5, 0.0, 3.140625
    np.testing.assert_array_equal(orc.to_f64(bits), [1.0, -2.5, 0.0, 3.140625])
    x = np.array([1.0, 1.00390625, 1.01171875, 3.14159, -1e-3, 0.0])
    ref = torch.tensor(x, dtype=torch.float64).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(orc.round_to_bf16(x), ref)
