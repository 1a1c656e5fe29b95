"""Pins for the oracle's confidence statistics and its Commit / Predict / Refill logic."""
import json
import math
import os

import numpy as np
import pytest
import scipy.special
import scipy.stats

from oracle import wedlm_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "alg1_hand_traces.json")


# ------------------------------------------------------------------ confidence: closed forms
def test_uniform_logits():
    V = 1001
    c = orc.confidence(np.full((1, V), 2.5))
    assert c["argmax"][0] == 0
    assert c["entropy"][0] == pytest.approx(math.log(V), rel=1e-13)
    assert c["maxprob"][0] == pytest.approx(1.0 / V, rel=1e-13)
    assert c["lse"][0] == pytest.approx(2.5 + math.log(V), rel=1e-13)


@pytest.mark.parametrize("a,V", [(3.0, 10), (12.0, 151936), (-4.0, 7)])
def test_one_hot_boost_closed_form(a, V):
    """logits (a, 0, ..., 0): p0 = e^a / (e^a + V - 1); H = -p0 ln p0 - (V-1) p1 ln p1."""
    x = np.zeros((1, V))
    x[0, 0] = a
    z = math.exp(a) + V - 1
    p0, p1 = math.exp(a) / z, 1.0 / z
    c = orc.confidence(x)
    assert c["entropy"][0] == pytest.approx(-p0 * math.log(p0) - (V - 1) * p1 * math.log(p1), rel=1e-12)
    assert c["maxprob"][0] == pytest.approx(max(p0, p1), rel=1e-12)
    assert c["argmax"][0] == (0 if a >= 0 else 1)
    assert c["lse"][0] == pytest.approx(math.log(z), rel=1e-12)


def test_ties_take_the_lowest_index_and_shift_invariance():
    x = np.array([[0.5, 2.0, -1.0, 2.0, 2.0]])
    c = orc.confidence(x)
    assert c["argmax"][0] == 1
    c2 = orc.confidence(x + 100.0)
    assert c2["argmax"][0] == 1
    assert c2["entropy"][0] == pytest.approx(c["entropy"][0], rel=1e-12)
    assert c2["maxprob"][0] == pytest.approx(c["maxprob"][0], rel=1e-12)
    assert c2["lse"][0] == pytest.approx(c["lse"][0] + 100.0, rel=1e-13)


def test_against_library_routines():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((5, 3000)) * 3.0
    x[2, 17] += 20.0           # a low-entropy row
    x[3] -= 1000.0             # large negative offset: underflowing terms contribute zero
    c = orc.confidence(x)
    for r in range(5):
        p = scipy.special.softmax(x[r])
        assert c["lse"][r] == pytest.approx(scipy.special.logsumexp(x[r]), rel=1e-13)
        assert c["entropy"][r] == pytest.approx(scipy.stats.entropy(p), rel=1e-10, abs=1e-14)
        assert c["maxprob"][r] == pytest.approx(p.max(), rel=1e-12)
        assert c["argmax"][r] == int(np.argmax(x[r]))
        assert 0.0 <= c["entropy"][r] <= math.log(3000) + 1e-12


def test_bf16_rows_are_widened_exactly():
    bits = np.array([[0x3F80, 0x4000, 0x4000, 0xBF80]], np.uint16)     # 1, 2, 2, -1
    c = orc.confidence(bits)
    ref = orc.confidence(np.array([[1.0, 2.0, 2.0, -1.0]]))
    assert c["argmax"][0] == 1 and c["entropy"][0] == ref["entropy"][0]


# ------------------------------------------------------------------ Algorithm 1, hand traces
def _cases():
    with open(GOLDEN) as f:
        return json.load(f)["cases"]


@pytest.mark.parametrize("case", _cases(), ids=lambda c: c["note"][:40])
def test_hand_worked_steps_of_algorithm_1(case):
    r = orc.select_commit_refill(
        case["tokens"], case["filled"], case["window_len"], case["prefix_len"],
        case["mask_argmax"], case["mask_entropy"], case["mask_maxprob"],
        conf_mode=case["conf_mode"], tau=case["tau"], lam=case["lam"], maxprob_thr=case["maxprob_thr"],
        mask_token_id=99, remaining_budget=case["budget"])
    assert r["committed_tokens"] == case["committed_tokens"]
    assert r["committed_count"] == len(case["committed_tokens"])
    assert r["filled_slots"] == case["filled_slots"]
    assert r["window_tokens"] == case["new_tokens"]
    assert r["filled"] == case["new_filled"]
    assert r["window_len"] == case["new_window_len"]
    assert r["prefix_len"] == case["new_prefix_len"]


# ------------------------------------------------------------------ reductions of the decision rule
def _run(H, lam, tau, filled=None):
    W = len(H)
    filled = [0] * W if filled is None else filled
    masks = [j for j in range(W) if not filled[j]]
    return orc.select_commit_refill(
        [99 if not f else 1 for f in filled], filled, W, 0, [10 + j for j in masks],
        [H[j] for j in masks], [0.5] * len(masks),
        conf_mode="entropy", tau=tau, lam=lam, maxprob_thr=0.9, mask_token_id=99)


def test_tau_plus_infinity_fills_every_mask():
    r = _run([3.0, 1.0, 2.0, 5.0], lam=0.0, tau=float("inf"))
    assert r["filled_slots"] == [0, 1, 2, 3]


def test_tau_minus_infinity_is_one_token_per_step_at_the_lowest_adjusted_entropy():
    r = _run([3.0, 1.0, 2.0, 0.95], lam=0.1, tau=float("-inf"))
    # adjusted: 3.0, 1.1, 2.2, 1.25 -> slot 1
    assert r["filled_slots"] == [1] and r["filled_count"] == 1


def test_huge_lambda_only_ever_selects_the_leftmost_mask():
    r = _run([0.2, 0.0, 0.0, 0.0], lam=1e9, tau=0.3, filled=[1, 0, 0, 0])
    # after committing slot 0 the leftmost mask is slot 1 (d = 0); every other mask is penalised away
    assert r["committed_count"] == 1 and r["filled_slots"] == [1]


def test_fallback_tie_goes_left():
    r = _run([1.0, 1.0, 1.0], lam=0.0, tau=0.1)
    assert r["filled_slots"] == [0]


# ------------------------------------------------------------------ the loop
def _toy_logits(V, seed):
    """A deterministic toy model: the logits of a slot depend on its position id and on the
    committed text only (so any decoding order must reproduce the same greedy text)."""
    def row(y, pos):
        h = (seed * 1000003 + pos * 7919 + sum((i + 1) * t for i, t in enumerate(y)) * 104729) % (2 ** 31)
        g = np.random.default_rng(h)
        return g.standard_normal(V) * 2.0
    return row


def test_window_of_one_is_greedy_one_token_at_a_time_decoding():
    V, P, N = 50, 3, 12
    row = _toy_logits(V, 1)

    def forward(y, toks, pos):
        return np.stack([row(y, p) for p in pos])

    out = orc.decode_loop(forward, prefix_len=P, window=1, max_new_tokens=N, conf_mode="entropy",
                          tau=0.3, lam=0.1, maxprob_thr=0.9, mask_token_id=V - 1)
    # independent greedy loop
    y = []
    for t in range(N):
        y.append(int(np.argmax(row(y, P + t))))
    assert out["y"] == y
    # W = 1 needs two forwards per token: one on the mask, one that commits the filled slot
    assert out["steps"] == 2 * N


@pytest.mark.parametrize("W,tau", [(4, 0.3), (8, 5.0), (3, float("-inf")), (16, 2.0)])
def test_loop_invariants(W, tau):
    V, P, N = 40, 5, 37
    rows = {}

    def forward(y, toks, pos):
        # logits depend on position only -> the final text is order independent
        out = []
        for p in pos:
            if p not in rows:
                rows[p] = np.random.default_rng(p).standard_normal(V) * (4.0 if p % 3 else 0.5)
            out.append(rows[p])
        return np.stack(out)

    out = orc.decode_loop(forward, prefix_len=P, window=W, max_new_tokens=N, conf_mode="entropy",
                          tau=tau, lam=0.05, maxprob_thr=0.9, mask_token_id=V - 1)
    assert len(out["y"]) == N
    assert out["y"] == [int(np.argmax(rows[P + t])) for t in range(N)]
    assert 0.0 < out["p_cache"] <= 1.0                       # Eq. 4
    assert out["n_fwd"] >= N
    assert out["steps"] >= math.ceil(N / W) + 1
    total = 0
    for tr in out["trace"]:
        total += tr["committed"]
        # position ids present in the window are exactly the next window_len logical positions
        assert sorted(tr["pos_ids"]) == list(range(P + total - tr["committed"], P + total - tr["committed"] + tr["window_len"]))
        assert tr["window_len"] <= W
    assert total == N
    # the window keeps its size until the budget runs out
    full = [tr["window_len"] for tr in out["trace"]]
    assert all(a >= b for a, b in zip(full, full[1:]))


def test_step_function_composes_the_parts():
    from workloads import get_config, make_step
    cfg = get_config("cfg1_tiny")
    inp = make_step(cfg)
    r = orc.step(inp, theta=cfg.rope_theta, conf_mode=cfg.conf_mode, tau=cfg.tau, lam=cfg.lam,
                 maxprob_thr=cfg.maxprob_thr, mask_token_id=cfg.mask_token_id, page_size=cfg.page_size)
    B, W = inp["filled"].shape
    assert r["out"].shape == inp["q"].shape
    for b in range(B):
        ps = r["per_seq"][b]
        assert ps["committed_count"] == r["n_commit"][b]
        assert ps["committed_tokens"] == inp["window_tokens"][b][: ps["committed_count"]].tolist()
        assert ps["filled_count"] >= 1 or r["n_filled"][b] == W
        assert ps["window_len"] == W


# ------------------------------------------------------------------ block-wise baseline
def test_block_wise_baseline_commits_all_or_nothing():
    """Hand-worked against the description of block decoding (Section 5.2, Fig. 2): [A,B,M,M] commits
    nothing although A,B lead the window; once the block is complete it is committed whole."""
    kw = dict(conf_mode="entropy", tau=0.5, lam=0.1, maxprob_thr=0.9, mask_token_id=99, block_commit=True)
    r = orc.select_commit_refill([11, 12, 99, 99], [1, 1, 0, 0], 4, 20, [7, 8], [0.1, 0.9], [0.9, 0.5], **kw)
    assert r["committed_count"] == 0 and r["committed_tokens"] == []
    assert r["window_tokens"] == [11, 12, 7, 99] and r["filled"] == [1, 1, 1, 0]
    assert r["prefix_len"] == 20 and r["window_len"] == 4
    r = orc.select_commit_refill([11, 12, 7, 9], [1, 1, 1, 1], 4, 20, [], [], [], **kw)
    assert r["committed_tokens"] == [11, 12, 7, 9] and r["prefix_len"] == 24
    assert r["window_tokens"] == [99, 99, 99, 99] and r["filled"] == [0, 0, 0, 0]
    ro = orc.reorder(np.array([[1, 1, 0, 0], [1, 1, 1, 1]], np.uint8), np.array([20, 20]), block_commit=True)
    assert ro["n_commit"].tolist() == [0, 4]


def test_block_wise_loop_produces_the_same_text():
    """With logits that depend on the position only, streaming and block-wise decoding write the same
    text; the block-wise loop commits in whole blocks only."""
    V, P, N, W = 40, 5, 33, 8
    rows = {}

    def forward(y, toks, pos):
        out = []
        for p in pos:
            if p not in rows:
                rows[p] = np.random.default_rng(p).standard_normal(V) * (4.0 if p % 3 else 0.5)
            out.append(rows[p])
        return np.stack(out)

    kw = dict(prefix_len=P, window=W, max_new_tokens=N, conf_mode="entropy", tau=2.0, lam=0.05, maxprob_thr=0.9,
              mask_token_id=V - 1)
    a = orc.decode_loop(forward, **kw)
    b = orc.decode_loop(forward, block_commit=True, **kw)
    assert a["y"] == b["y"] and len(a["y"]) == N
    assert all(tr["committed"] in (0, tr["window_len"]) for tr in b["trace"])
    assert any(0 < tr["committed"] < tr["window_len"] for tr in a["trace"])
