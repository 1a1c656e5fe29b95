"""Pins for the oracle's Sample() at a temperature (Algorithm 1, "W[i] <- Sample(l_i)"; Section 6.1
evaluates at temperature 0.1).

The sampler is pinned to facts outside itself: the Gumbel-max identity (its draws must follow
softmax(l / T), which a wrong sign, a temperature applied the wrong way round or a biased uniform
all break), the T -> 0 limit (greedy arg-max), number theory (the integer mixer must be a bijection,
shown by inverting it with modular inverses), and the statistical quality of the stateless uniforms
across the three counters (token, position, sequence)."""
import numpy as np

from oracle import wedlm_oracle as orc
from workloads import synth


def _chi2(counts, expected):
    counts, expected = np.asarray(counts, float), np.asarray(expected, float)
    return float(np.sum((counts - expected) ** 2 / expected))


def test_mixer_is_a_bijection():
    # invert each step: x ^= x >> k is undone by repeating the shift-xor; an odd multiply by its inverse mod 2^32
    def unxorshift(x, k):
        y = x.copy()
        for _ in range(32 // k + 1):
            y = x ^ (y >> np.uint32(k))
        return y

    g = np.random.default_rng(1)
    x = g.integers(0, 2 ** 32, size=200_000, dtype=np.uint64).astype(np.uint32)
    y = orc.mix32(x)
    inv1 = np.uint32(pow(0x7FEB352D, -1, 2 ** 32))
    inv2 = np.uint32(pow(0x846CA68B, -1, 2 ** 32))
    with np.errstate(over="ignore"):
        z = unxorshift(y, 16)
        z = z * inv2
        z = unxorshift(z, 15)
        z = z * inv1
        z = unxorshift(z, 16)
    assert np.array_equal(z, x)
    assert len(np.unique(y)) == len(np.unique(x))


def test_uniforms_are_uniform_and_uncorrelated_along_every_counter():
    V = 1 << 16
    u = orc.sample_uniforms(orc.sample_key(11, 22, 3, 77), V)
    assert 0.0 < u.min() and u.max() < 1.0
    assert abs(u.mean() - 0.5) < 4 * np.sqrt(1 / 12 / V)
    assert abs(u.var() - 1 / 12) < 2e-3
    counts = np.bincount((u * 64).astype(int), minlength=64)
    assert _chi2(counts, np.full(64, V / 64)) < 120.0            # df = 63, far tail
    # neighbours along the token counter
    assert abs(np.corrcoef(u[:-1], u[1:])[0, 1]) < 0.02
    # the same tokens under neighbouring positions / sequences / seeds
    for other in (orc.sample_key(11, 22, 3, 78), orc.sample_key(11, 22, 4, 77), orc.sample_key(12, 22, 3, 77),
                  orc.sample_key(11, 23, 3, 77)):
        u2 = orc.sample_uniforms(other, V)
        assert abs(np.corrcoef(u, u2)[0, 1]) < 0.02
        assert np.mean(u == u2) < 1e-3


def test_draws_follow_softmax_at_temperature():
    # Gumbel-max identity: P(token = v) = softmax(l / T)_v
    logits = np.array([1.0, 0.2, -0.5, 0.9, -2.0, 0.0], np.float32)
    for T in (0.7, 0.1 * 5, 2.0):
        p = np.exp(logits.astype(np.float64) / T)
        p /= p.sum()
        n = 60_000
        counts = np.zeros(len(logits))
        for r in range(n):
            tok, _ = orc.sample_token(logits, T, (2024, 7), r % 13, r)
            counts[tok] += 1
        assert _chi2(counts, p * n) < 25.0, (T, counts / n, p)    # df = 5: P(chi2 > 25) ~ 1e-4


def test_flat_logits_give_uniform_independent_tokens():
    V, n = 8, 40_000
    flat = np.zeros(V, np.float32)
    toks = np.array([orc.sample_token(flat, 1.0, (5, 6), 0, pos)[0] for pos in range(n)])
    assert _chi2(np.bincount(toks, minlength=V), np.full(V, n / V)) < 30.0       # df = 7
    joint = np.zeros((V, V))
    np.add.at(joint, (toks[:-1], toks[1:]), 1)
    assert _chi2(joint.reshape(-1), np.full(V * V, (n - 1) / V / V)) < 120.0     # df = 63


def test_small_temperature_is_greedy():
    g = np.random.default_rng(3)
    for r in range(200):
        x = g.standard_normal(500).astype(np.float32)
        a = int(np.argmax(x))
        x[a] += 0.5                                   # clear lead; at T = 1e-3 the lead is worth 500
        tok, margin = orc.sample_token(x, 1e-3, (9, 9), r, 3 * r)
        assert tok == a and margin > 100.0


def test_draw_depends_only_on_seed_sequence_and_position():
    g = np.random.default_rng(4)
    x = g.standard_normal(3000).astype(np.float32)
    base = orc.sample_token(x, 1.0, (1, 2), 5, 100)
    assert orc.sample_token(x.copy(), 1.0, (1, 2), 5, 100) == base
    others = [orc.sample_token(x, 1.0, s, b, p)[0] for s, b, p in
              [((1, 2), 5, 101), ((1, 2), 6, 100), ((1, 3), 5, 100), ((2, 2), 5, 100), ((1, 2), 5, 99)]]
    assert sum(o != base[0] for o in others) >= 4     # flat-ish distribution: a repeat is a 1-in-thousands event


def test_step_with_temperature_fills_sampled_tokens_and_keeps_confidences():
    cfg = synth.CONFIGS["cfg1_tiny"]
    inp = synth.make_step(cfg, seed=synth.BASE_SEED, with_logits=True)
    kw = dict(theta=cfg.rope_theta, conf_mode="entropy", tau=50.0, lam=0.0, maxprob_thr=0.9,
              mask_token_id=cfg.mask_token_id, page_size=cfg.page_size, with_attention=False)
    greedy = orc.step(inp, **kw)
    hot = orc.step(inp, temperature=5.0, sample_seed=(77, 88), **kw)
    # confidences come from the raw logits either way
    for key in ("entropy", "maxprob", "lse", "argmax"):
        assert np.array_equal(np.nan_to_num(greedy[key], nan=-1.0), np.nan_to_num(hot[key], nan=-1.0))
    differ = 0
    for b in range(cfg.batch):
        nf = int(hot["n_filled"][b])
        for i in range(nf, cfg.window):
            j = int(hot["perm"][b, i])
            want, _ = orc.sample_token(inp["logits"][b, i], 5.0, (77, 88), b, int(inp["prefix_len"][b]) + j)
            assert hot["sampled"][b, i] == want
            differ += int(want != greedy["argmax"][b, i])
        # tau = 50 selects every mask: the window after the step carries exactly the sampled tokens
        r = hot["per_seq"][b]
        n = r["committed_count"]
        for k, j in enumerate(r["mask_slots"]):
            if j >= n:
                assert r["window_tokens"][j - n] == hot["sampled"][b, nf + k]
    assert differ > 0            # at T = 5 over ~1000 tokens the draw is essentially never the arg-max everywhere
