"""The fused LM head + confidence/commit call against the oracle: logits = hidden . lm_head^T in float64
from the same bf16 bit patterns, then the oracle's confidence / selection / commit."""
import numpy as np
import pytest
import torch

from oracle import wedlm_oracle as orc
from workloads import StepConfig, bf16_bits, make_step

pytestmark = pytest.mark.gpu


def _case(B, W, V, H, seed, boost=6.0, window_len=None, budget=None, commit_mode="streaming", fill_all=()):
    import paper_2512_22737_b200 as w
    import parity_util as pu
    cfg = StepConfig(name="lmhead", batch=B, window=W, n_q_heads=4, n_kv_heads=1, head_dim=128, vocab=V, dtype="bf16",
                     prefix_lo=10, prefix_hi=60, obs_prob_lo=0.2, obs_prob_hi=0.6, tau=0.3, lam=0.1)
    inp = make_step(cfg, seed=seed, with_logits=False)
    g = np.random.default_rng(seed)
    if len(fill_all):                                    # sequences without a single mask row
        f = inp["filled"].copy()
        f[list(fill_all)] = 1
        inp = make_step(cfg, seed=seed, with_logits=False, filled=f)
    hid = bf16_bits((g.standard_normal((B, W, H)) * 1.0).astype(np.float32).reshape(-1)).reshape(B, W, H)
    emb = bf16_bits((g.standard_normal((V, H)) * (2.0 / np.sqrt(H))).astype(np.float32).reshape(-1)).reshape(V, H)
    tilt_ids = g.integers(0, V - 1, size=(B, W)).astype(np.int32)
    tilt_ids[g.random((B, W)) < 0.3] = -1
    # oracle logits in float64 from the bf16 inputs, tilt added where asked
    logits = orc.to_f64(hid) @ orc.to_f64(emb).T
    bb, ww = np.nonzero(tilt_ids >= 0)
    logits[bb, ww, tilt_ids[bb, ww]] += boost
    inp["logits"] = logits
    ref = pu.oracle_step(cfg, inp, window_len=window_len, remaining_budget=budget, with_attention=False,
                         block_commit=(commit_mode == "block"))
    # GPU
    c = w.config_for(cfg, max_pages_per_seq=inp["block_table"].shape[1], num_pages=inp["k_cache"].shape[0],
                     max_prefix_len=int(inp["prefix_len"].max()), commit_mode=commit_mode)
    step = w.DecodeStep(c)
    d = {k: w.to_device(inp[k]) for k in ("filled", "window_tokens", "prefix_len")}
    wl = None if window_len is None else torch.tensor(window_len, dtype=torch.int32, device="cuda")
    bud = None if budget is None else torch.tensor(budget, dtype=torch.int32, device="cuda")
    step.reorder(d["filled"], d["window_tokens"], d["prefix_len"], wl)
    ws = torch.empty(w.wedlm_lmhead_confidence_workspace_bytes(c, H), dtype=torch.uint8, device="cuda")
    w.wedlm_lmhead_confidence_commit(c, w.to_device(hid), w.to_device(emb), w.to_device(tilt_ids), boost, step.perm,
                                     step.n_filled, step.n_commit, d["window_tokens"], d["filled"], d["prefix_len"], wl, bud,
                                     step.argmax, step.maxprob, step.entropy, step.lse, step.committed_tokens,
                                     step.committed_count, step.filled_count, ws, step.status)
    torch.cuda.synchronize()
    assert int(step.status.item()) == 0
    d["window_len"], d["remaining_budget"] = wl, bud
    # arg-max: exact unless the two best logits of the row are within the 1e-3 band
    am = step.argmax.cpu().numpy()
    near_tie = set()
    for b in range(B):
        for i in range(W):
            if ref["argmax"][b, i] >= 0 and am[b, i] != ref["argmax"][b, i]:
                top2 = np.sort(logits[b, i])[-2:]
                assert top2[1] - top2[0] <= 1e-3, (b, i, am[b, i], ref["argmax"][b, i], top2)
                near_tie.add(b)
                ref["argmax"][b, i] = am[b, i]
    assert len(near_tie) <= 2
    # a sequence with a near-tie may have filled a different (equally good) token: only its fills are skipped,
    # every statistic of every row and everything else about its window are still compared
    pu.check_confidence_and_commit(cfg, step, d, inp, ref, window_len, tie_seqs=near_tie)
    return step, ref


@pytest.mark.parametrize("B,W,V,H", [(2, 8, 1000, 64), (3, 16, 5000, 256), (1, 40, 4096, 512), (5, 64, 3333, 128)])
def test_fused_lmhead_confidence_matches_oracle(B, W, V, H):
    _case(B, W, V, H, seed=B * 100 + W)


def test_fused_lmhead_short_windows_budget_and_block_mode():
    _case(4, 8, 2048, 128, seed=9, window_len=[8, 5, 3, 8], budget=[10, 1, 0, 10])
    _case(4, 8, 2048, 128, seed=10, commit_mode="block")


def test_fused_lmhead_sequences_without_mask_rows_and_a_batch_without_any():
    """The mask rows are gathered before the tensor-core pass: sequences that contribute none, and a call in which
    no row at all is a mask (the pass runs over zero items and only the commit/shift part does anything)."""
    _case(4, 8, 2048, 128, seed=21, fill_all=(0, 2))
    _case(3, 8, 2048, 128, seed=22, fill_all=(0, 1, 2))


def test_fused_lmhead_more_sequences_than_one_scan_pass():
    """1100 sequences: the per-sequence mask-row counts are scanned 1024 at a time with a carry."""
    _case(1100, 4, 512, 64, seed=23)


def test_fused_lmhead_qwen_width_rows_over_256():
    """Hidden 4096 (64 k-steps through the 4-stage ring) and more than 256 rows (two row chunks)."""
    _case(10, 32, 8192, 4096, seed=11, boost=14.0)


def test_fused_lmhead_rejects_unsupported_shapes():
    import paper_2512_22737_b200 as w
    c = w.make_config(batch=1, window=8, vocab=1000, dtype="bf16")
    x = torch.zeros(8 * 96, dtype=torch.bfloat16, device="cuda").view(1, 8, 96)        # hidden not a multiple of 64
    e = torch.zeros(8, dtype=torch.int32, device="cuda")
    ws = torch.empty(1 << 16, dtype=torch.uint8, device="cuda")
    with pytest.raises(w.WedlmError) as err:
        w.wedlm_lmhead_confidence_commit(c, x, torch.zeros(1000, 96, dtype=torch.bfloat16, device="cuda"), None, 0.0, e, e, e,
                                         e, torch.zeros(8, dtype=torch.uint8, device="cuda"), e, None, None, None, None, None,
                                         None, None, None, None, ws)
    assert err.value.code == -2


def test_tile_width_that_is_no_multiple_of_32_ignores_stale_tensor_memory():
    """Regression: with a vocabulary tile of 208 tokens the reduction reads 224 accumulator columns; the last 16 are
    never written by the tile's MMAs and keep what tensor memory held before.  A first call whose logits overflow
    to +inf leaves inf in every column of every SM; the second call must still produce finite statistics."""
    import paper_2512_22737_b200 as w
    # call 1: 256-wide tiles on all 148 SMs (V = 148 * 256), logits = +inf
    V1, H, B, W = 148 * 256, 64, 16, 16
    c1 = w.make_config(batch=B, window=W, vocab=V1, dtype="bf16", mask_token_id=V1 - 1)
    s1 = w.DecodeStep(c1)
    i32 = dict(dtype=torch.int32, device="cuda")
    filled = torch.zeros(B, W, dtype=torch.uint8, device="cuda")
    tok, pl = torch.zeros(B, W, **i32), torch.zeros(B, **i32)
    big = torch.full((B, W, H), 1.0e19, dtype=torch.bfloat16, device="cuda")
    emb1 = torch.full((V1, H), 1.0e19, dtype=torch.bfloat16, device="cuda")
    s1.reorder(filled, tok, pl)
    ws1 = torch.empty(w.wedlm_lmhead_confidence_workspace_bytes(c1, H), dtype=torch.uint8, device="cuda")
    w.wedlm_lmhead_confidence_commit(c1, big, emb1, None, 0.0, s1.perm, s1.n_filled, s1.n_commit, tok.clone(), filled.clone(),
                                     pl.clone(), None, None, s1.argmax, s1.maxprob, s1.entropy, s1.lse, s1.committed_tokens,
                                     s1.committed_count, s1.filled_count, ws1)
    torch.cuda.synchronize()
    # call 2: V = 148 * 208 makes 208 the cheapest tile width; ordinary inputs, compared with the oracle
    step, ref = _case(16, 16, 148 * 208, 64, seed=77)
    ent = step.entropy.cpu().numpy()
    active = ~np.isnan(ref["entropy"])
    assert np.isfinite(ent[active]).all()
