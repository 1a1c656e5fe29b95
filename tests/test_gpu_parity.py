"""GPU-vs-oracle parity of the whole step, through the C-ABI binding.

Small cases and the full-size serving and long-context workloads alike are compared element by
element: every integer output, every confidence row, every attention output vector."""
import numpy as np
import pytest
import torch

from workloads import get_config, make_step
from oracle import wedlm_oracle as orc

pytestmark = pytest.mark.gpu

IMPLS = ["generic", "tensor"]


def _small_qwen(**kw):
    base = get_config("cfg2_qwen_b1").replace(vocab=20000)
    return base.replace(**kw)


@pytest.mark.parametrize("seed", [251222737, 1, 2])
def test_cfg1_tiny_fp32(seed):
    import parity_util as pu
    cfg = get_config("cfg1_tiny")
    r = pu.full_parity(cfg, make_step(cfg, seed=seed))
    assert r["attn_err"] < 1e-4          # fp32 end to end


def test_cfg1_tiny_with_boost_exercises_the_threshold_branch():
    import parity_util as pu
    cfg = get_config("cfg1_tiny").replace(boost=12.0, boost_prob=0.6)
    for seed in (3, 4, 5):
        r = pu.full_parity(cfg, make_step(cfg, seed=seed))
        assert r["attn_err"] < 1e-4


@pytest.mark.parametrize("impl", IMPLS)
def test_cfg2_qwen_single_sequence(impl):
    import parity_util as pu
    cfg = get_config("cfg2_qwen_b1")
    r = pu.full_parity(cfg, make_step(cfg), attn_impl=impl)
    print("cfg2 attention error", r["attn_err"], "excluded", r["excluded"])


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("boost", [14.4, 16.4, 20.4])
def test_cfg2_calibrated_boosts_mixed_decisions(impl, boost):
    """Boosts near 12.4 + s put rows on either side of tau = 0.3 (the literal +8 never passes)."""
    import parity_util as pu
    cfg = get_config("cfg2_qwen_b1").replace(boost=boost, boost_prob=0.7)
    r = pu.full_parity(cfg, make_step(cfg, seed=11), attn_impl=impl)
    assert r["excluded"] <= 1


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("B,W,lo,hi", [(3, 16, 0, 40), (4, 32, 100, 700), (2, 64, 1000, 1100), (5, 5, 1, 300), (2, 1, 17, 17)])
def test_ragged_batches_span_tiles_and_tails(impl, B, W, lo, hi):
    import parity_util as pu
    cfg = _small_qwen(batch=B, window=W, prefix_lo=lo, prefix_hi=hi, obs_prob_lo=0.1, obs_prob_hi=0.7,
                      boost=12.0, boost_prob=0.5, name="ragged")
    pu.full_parity(cfg, make_step(cfg, seed=B * 100 + W), attn_impl=impl)


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("Hq,Hkv,D", [(4, 4, 64), (8, 1, 128), (2, 1, 32), (6, 2, 256)])
def test_head_geometries(impl, Hq, Hkv, D):
    import parity_util as pu
    cfg = _small_qwen(batch=2, window=8, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, prefix_lo=5, prefix_hi=90,
                      vocab=3000, name="heads")
    pu.full_parity(cfg, make_step(cfg, seed=Hq * 7 + D), attn_impl="generic")


@pytest.mark.parametrize("Hq,Hkv,W", [(8, 8, 40), (8, 4, 70), (16, 2, 20), (16, 1, 9), (4, 4, 130)])
def test_tensor_path_group_sizes(Hq, Hkv, W):
    """G = 1, 2, 8, 16 with D = 128: the 128-row tile holds 128/G window slots; windows that need one,
    two (partial) or more row tiles."""
    import parity_util as pu
    cfg = _small_qwen(batch=2, window=W, n_q_heads=Hq, n_kv_heads=Hkv, prefix_lo=200, prefix_hi=400, vocab=2048,
                      name="groups")
    inp = make_step(cfg, seed=Hq * 100 + Hkv)
    r = pu.full_parity(cfg, inp, attn_impl="tensor")
    assert r["attn_err"] <= pu.ATTN_REL_TOL


@pytest.mark.parametrize("W", [128, 1024])
def test_large_windows(W):
    """Window sizes up to the maximum the ABI accepts (generic path at 1024, both paths at 128)."""
    import parity_util as pu
    cfg = _small_qwen(batch=1, window=W, n_q_heads=4, n_kv_heads=1, prefix_lo=50, prefix_hi=50, vocab=512,
                      name="bigwindow")
    inp = make_step(cfg, seed=W)
    pu.full_parity(cfg, inp, attn_impl="generic" if W > 128 else "tensor")


@pytest.mark.parametrize("W,P", [(512, 700), (1024, 3000)])
def test_many_row_tiles_share_the_runs_of_one_key_stream(W, P):
    """Tensor path with 16 and 32 row tiles per key stream: every run of key tiles is taken by one CTA per row tile,
    and the row tiles of the early window slots, whose horizon ends sooner, skip the last runs."""
    import parity_util as pu
    cfg = _small_qwen(batch=2, window=W, n_q_heads=4, n_kv_heads=1, prefix_lo=P, prefix_hi=P + 200, vocab=512,
                      name="manytiles")
    inp = make_step(cfg, seed=W + P)
    res = pu.full_parity(cfg, inp, attn_impl="tensor")
    assert int(res["step"].status.item()) == 0


def test_long_ragged_sequences_whose_runs_cross_from_one_key_stream_into_the_next():
    """Few work units and long prefixes: the tensor path cuts the key tiles of all (sequence, KV head) streams into
    equal runs, here of about 35 tiles, so most CTAs finish one stream and start the next (another head, or another
    sequence of different length), with two row tiles per stream sharing every run."""
    import parity_util as pu
    cfg = _small_qwen(batch=3, window=48, n_q_heads=8, n_kv_heads=2, prefix_lo=50000, prefix_hi=60000, vocab=512,
                      name="crossing")
    inp = make_step(cfg, seed=4848, prefix_len=np.array([60000, 50003, 55017], dtype=np.int32))
    res = pu.full_parity(cfg, inp, attn_impl="tensor")
    assert int(res["step"].status.item()) == 0


def test_one_long_sequence_is_spread_over_every_cta_slot():
    """A single sequence of 150 000 cached tokens: its 8 key streams are cut into about 37 pieces each (close to the
    number of partial slots the workspace provides per row), one run per CTA slot, runs crossing from one KV head
    into the next."""
    import parity_util as pu
    cfg = _small_qwen(batch=1, window=16, prefix_lo=150000, prefix_hi=150000, vocab=512, name="one_long")
    inp = make_step(cfg, seed=150)
    res = pu.full_parity(cfg, inp, attn_impl="tensor")
    assert int(res["step"].status.item()) == 0


@pytest.mark.parametrize("P", [0, 1, 15, 16, 17, 31, 33])
def test_page_boundaries(P):
    import parity_util as pu
    cfg = _small_qwen(batch=1, window=24, prefix_lo=P, prefix_hi=P, vocab=1000, name="pages")
    pu.full_parity(cfg, make_step(cfg, seed=P), attn_impl="generic")


def test_degenerate_windows():
    import parity_util as pu
    cfg = _small_qwen(batch=3, window=16, prefix_lo=30, prefix_hi=60, vocab=5000, name="degenerate")
    inp = make_step(cfg, seed=9)
    for pattern in (np.ones((3, 16), np.uint8), np.zeros((3, 16), np.uint8)):
        inp2 = make_step(cfg, seed=9, filled=pattern)
        pu.full_parity(cfg, inp2)
    # leading run then a gap
    f = np.zeros((3, 16), np.uint8)
    f[:, :5] = 1
    f[:, 7:9] = 1
    pu.full_parity(cfg, make_step(cfg, seed=9, filled=f))


def test_short_windows_and_budget():
    import parity_util as pu
    cfg = _small_qwen(batch=4, window=8, prefix_lo=10, prefix_hi=50, vocab=2000, boost=14.0, boost_prob=0.8,
                      name="short")
    f = np.array([[1, 1, 0, 1, 0, 0, 1, 1], [1, 1, 1, 1, 1, 0, 0, 0], [0, 1, 1, 0, 0, 0, 0, 0], [1, 1, 1, 0, 0, 0, 0, 0]], np.uint8)
    inp = make_step(cfg, seed=21, filled=f)
    pu.full_parity(cfg, inp, window_len=[8, 5, 3, 3], remaining_budget=[100, 2, 0, 1])


def test_step_wise_scheme_fills_exactly_the_lowest_adjusted_entropy():
    """tau = -inf: no mask ever passes Eq. 11, so every step fills the single mask with the lowest H + lambda d
    (the unified step-wise scheme of Section 6.1, W = 6, lambda = 0.1)."""
    import parity_util as pu
    cfg = _small_qwen(batch=5, window=6, prefix_lo=30, prefix_hi=400, vocab=4096, tau=float("-inf"), lam=0.1, boost=9.0,
                      boost_prob=0.5, name="stepwise")
    for seed in (51, 52):
        r = pu.full_parity(cfg, make_step(cfg, seed=seed))
        fc = r["step"].filled_count.cpu().numpy()
        n_mask = cfg.window - r["ref"]["n_filled"]
        assert ((fc == 1) | (n_mask == 0)).all()


def test_maxprob_mode_bf16():
    import parity_util as pu
    cfg = _small_qwen(batch=2, window=16, prefix_lo=40, prefix_hi=80, vocab=4096, conf_mode="maxprob",
                      maxprob_thr=0.9, boost=13.0, boost_prob=0.6, name="maxprob")
    pu.full_parity(cfg, make_step(cfg, seed=31))


def test_unaligned_vocab_takes_the_scalar_path():
    import parity_util as pu
    cfg = _small_qwen(batch=2, window=8, prefix_lo=20, prefix_hi=20, vocab=10007, boost=11.0, name="oddvocab")
    pu.full_parity(cfg, make_step(cfg, seed=41))


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("W,P", [(16, 100), (40, 333), (64, 64), (5, 1000), (1, 31), (32, 0), (33, 4097)])
def test_window_sizes_and_row_tiles(impl, W, P):
    """W*G below, equal to and above one 128-row tile, partial second tile, chunk boundaries."""
    import parity_util as pu
    cfg = _small_qwen(batch=2, window=W, prefix_lo=P, prefix_hi=P + 70, vocab=2048, name="rowtiles")
    pu.full_parity(cfg, make_step(cfg, seed=W * 1000 + P), attn_impl=impl)


@pytest.mark.parametrize("impl", IMPLS)
def test_stale_cache_rows_beyond_the_window_cannot_leak(impl):
    """Rows of the last page past P + W may hold anything (here NaN and Inf bit patterns); they are
    masked by index, so the outputs must not change."""
    import parity_util as pu
    cfg = _small_qwen(batch=2, window=8, prefix_lo=70, prefix_hi=70, vocab=2048, name="stale")
    inp = make_step(cfg, seed=77)
    ref = pu.oracle_step(cfg, inp)
    B, W = inp["filled"].shape
    for b in range(B):
        P = int(inp["prefix_len"][b])
        for t in range(P + W, ((P + W + 15) // 16) * 16):
            pg = inp["block_table"][b, t // 16]
            inp["k_cache"][pg, :, t % 16, :] = 0x7FC0       # NaN
            inp["v_cache"][pg, :, t % 16, :] = 0x7F80       # +Inf
    # every spare / unowned page too
    owned = set(inp["block_table"][inp["block_table"] >= 0].tolist())
    for pg in range(inp["k_cache"].shape[0]):
        if pg not in owned:
            inp["k_cache"][pg] = 0x7FC0
            inp["v_cache"][pg] = 0x7FC0
    step, d = pu.run_gpu_step(cfg, inp, attn_impl=impl)
    got = pu.bf16_from_device(step.out)
    assert np.isfinite(got).all()
    assert pu.attn_vector_error(got, ref["out"]).max() <= pu.ATTN_REL_TOL


@pytest.mark.parametrize("where,factor", [(300, 40.0), (0, 40.0), (599, 25.0), (300, 6.0)])
def test_outlier_keys_move_the_running_maximum_by_large_steps(where, factor):
    """A cache page scaled up so that its scores lie tens of powers of two above (or below) everything else.
    With N(0,1) data a row's running maximum creeps up by a bit or two over a whole prefix, so the branch of
    the tensor path that rescales its accumulator (taken when the maximum grows by more than 2^8) never runs;
    here it runs in the middle of the prefix, right after the first tile, and on the last tile.  Scores that
    large multiply the effect of the bf16 rounding of the rotated q by the same factor, so the fp64 oracle is
    not the right yardstick; the CUDA-core path is: it reads the same rounded q and the same cache, computes
    the softmax in fp32 and rescales on every page."""
    import parity_util as pu
    from workloads import bf16_bits, bf16_to_f32
    cfg = _small_qwen(batch=2, window=16, prefix_lo=600, prefix_hi=600, vocab=1024, name="outlier")
    inp = make_step(cfg, seed=int(where + factor))
    for b in range(2):
        pg = inp["block_table"][b, (where + 16 * b) // 16]
        page = bf16_to_f32(inp["k_cache"][pg].reshape(-1)) * np.float32(factor)
        inp["k_cache"][pg] = bf16_bits(page).reshape(inp["k_cache"][pg].shape)
    outs = {}
    for impl in IMPLS:
        step, _ = pu.run_gpu_step(cfg, inp, attn_impl=impl)
        assert int(step.status.item()) == 0
        outs[impl] = pu.bf16_from_device(step.out)
        assert np.isfinite(outs[impl]).all()
    assert pu.attn_vector_error(outs["tensor"], outs["generic"]).max() <= pu.ATTN_REL_TOL


def test_tensor_path_refuses_shapes_it_does_not_cover():
    import paper_2512_22737_b200 as w
    cfg = w.make_config(batch=1, window=8, n_q_heads=4, n_kv_heads=2, head_dim=64, max_pages_per_seq=8,
                        num_pages=8, max_prefix_len=64, attn_impl="tensor")
    t = torch.zeros(4096, dtype=torch.bfloat16, device="cuda")
    i = torch.zeros(64, dtype=torch.int32, device="cuda")
    ws = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    with pytest.raises(w.WedlmError) as e:
        w.wedlm_window_attn(cfg, t, t, t, t, t, i, i, i, t, None, ws)
    assert e.value.code == -2


def test_empty_batch_is_a_noop():
    import paper_2512_22737_b200 as w
    cfg = w.make_config(batch=0, window=8, n_q_heads=4, n_kv_heads=2, head_dim=64, max_pages_per_seq=4,
                        num_pages=4, vocab=100)
    e = torch.empty(0, dtype=torch.int32, device="cuda")
    w.wedlm_reorder(cfg, torch.empty(0, dtype=torch.uint8, device="cuda"), None, e, None, e, e, e, None, e, e)
    torch.cuda.synchronize()


def test_bad_block_table_sets_status_and_does_not_fault():
    import paper_2512_22737_b200 as w
    import parity_util as pu
    cfg = _small_qwen(batch=2, window=8, prefix_lo=40, prefix_hi=40, vocab=1000, name="badpage")
    inp = make_step(cfg, seed=5)
    inp["block_table"][1, 1] = inp["k_cache"].shape[0] + 7        # outside the pool
    step, d = pu.run_gpu_step(cfg, inp)
    assert int(step.status.item()) & w.binding.WEDLM_STATUS_BAD_PAGE
    assert torch.isfinite(step.out.float()).all()
    # the untouched sequence is still right
    inp_ok = make_step(cfg, seed=5)
    ref = pu.oracle_step(cfg, inp_ok)
    err = pu.attn_vector_error(pu.bf16_from_device(step.out)[0], ref["out"][0])
    assert err.max() <= pu.ATTN_REL_TOL


def test_kv_append_alone_and_window_refill_alone():
    import paper_2512_22737_b200 as w
    import parity_util as pu
    cfg = _small_qwen(batch=3, window=8, prefix_lo=10, prefix_hi=70, vocab=1000, name="append")
    inp = make_step(cfg, seed=6)
    d = pu.device_inputs(inp)
    c = w.config_for(cfg, max_pages_per_seq=inp["block_table"].shape[1], num_pages=inp["k_cache"].shape[0],
                     max_prefix_len=int(inp["prefix_len"].max()))
    ro = orc.reorder(inp["filled"], inp["prefix_len"])
    pos = torch.tensor(ro["pos_ids"], dtype=torch.int32, device="cuda")
    count = torch.tensor([8, 3, 0], dtype=torch.int32, device="cuda")
    slots = torch.empty(3, 8, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    k_before = d["k_cache"].clone()
    w.wedlm_kv_append(c, d["k"], d["v"], pos, d["k_cache"], d["v_cache"], d["block_table"], d["prefix_len"], count,
                      slots, status)
    torch.cuda.synchronize()
    want_slots = orc.stage_slots(inp["block_table"], inp["prefix_len"], 8, cfg.page_size)
    want_slots[1, 3:] = -1
    want_slots[2, :] = -1
    np.testing.assert_array_equal(slots.cpu().numpy(), want_slots)
    k_rot = orc.rope(orc.to_f64(inp["k"]), ro["pos_ids"][:, :, None], cfg.rope_theta)
    kc = pu.bf16_from_device(d["k_cache"])
    changed = (d["k_cache"] != k_before).any(dim=(1, 3)).sum().item()
    assert changed <= 11 * cfg.n_kv_heads
    for b, n in ((0, 8), (1, 3)):
        for i in range(n):
            s = int(want_slots[b, i])
            got = kc[s // 16, :, s % 16]
            want = orc.round_to_bf16(k_rot[b, i])
            assert (np.abs(got - want) <= np.abs(want) * 2.0 ** -7 + np.abs(orc.to_f64(inp["k"][b, i])).max() * 2.0 ** -20).all()
    # refill alone
    n_commit = torch.tensor(ro["n_commit"], dtype=torch.int32, device="cuda")
    ct = torch.empty(3, 8, dtype=torch.int32, device="cuda")
    cc = torch.empty(3, dtype=torch.int32, device="cuda")
    w.wedlm_window_refill(c, n_commit, d["window_tokens"], d["filled"], d["prefix_len"], None, None, ct, cc)
    torch.cuda.synchronize()
    for b in range(3):
        n = int(ro["n_commit"][b])
        assert cc[b].item() == n
        assert ct[b, :n].cpu().tolist() == inp["window_tokens"][b, :n].tolist()
        want_tok = inp["window_tokens"][b, n:].tolist() + [cfg.mask_token_id] * n
        want_fil = inp["filled"][b, n:].tolist() + [0] * n
        assert d["window_tokens"][b].cpu().tolist() == want_tok
        assert d["filled"][b].cpu().tolist() == want_fil
        assert d["prefix_len"][b].item() == inp["prefix_len"][b] + n


_FULL_SIZE_REF = {}


def _full_size_reference(cfg_name):
    """Inputs and the oracle's whole step (attention of every row included) of a full-size workload,
    computed once per test session and shared by the two attention implementations."""
    import parity_util as pu
    if cfg_name not in _FULL_SIZE_REF:
        cfg = get_config(cfg_name)
        inp = make_step(cfg)
        _FULL_SIZE_REF[cfg_name] = (cfg, inp, pu.oracle_step(cfg, inp, with_attention=True))
    return _FULL_SIZE_REF[cfg_name]


def _full_size(cfg_name, impl):
    """The benchmark's own workload at its full size, in the launch configuration the benchmark times:
    every integer output, every confidence row, every attention output vector (all B*W*Hq of them) and
    every staged cache row are compared with the oracle."""
    import parity_util as pu
    cfg, inp, ref = _full_size_reference(cfg_name)
    step, d = pu.run_gpu_step(cfg, inp, attn_impl=impl)
    pu.check_reorder(step, ref)
    worst = pu.check_attention(cfg, step, d, inp, ref)
    excluded = pu.check_confidence_and_commit(cfg, step, d, inp, ref)
    print(cfg_name, impl, "worst attention error over all vectors", worst, "excluded sequences", excluded)


@pytest.mark.parametrize("impl", IMPLS)
def test_cfg3_batched_serving_full_size_every_vector(impl):
    _full_size("cfg3_batched", impl)


@pytest.mark.parametrize("impl", IMPLS)
def test_cfg4_long_context_full_size_every_vector(impl):
    _full_size("cfg4_long", impl)


def test_reorder_all_1024_patterns_of_a_10_slot_window_in_one_launch():
    """Every fill pattern of W = 10 as one batch of 1024 sequences: permutation, inverse, position ids,
    scattered tokens, filled count and commit length bit-exact against the oracle (Eq. 5-6, Algorithm 1)."""
    import itertools
    import paper_2512_22737_b200 as w
    W = 10
    pats = np.array(list(itertools.product([0, 1], repeat=W)), dtype=np.uint8)
    B = len(pats)
    rng = np.random.default_rng(10)
    P = rng.integers(0, 5000, size=B).astype(np.int32)
    toks = rng.integers(0, 150000, size=(B, W)).astype(np.int32)
    for window_len in (None, rng.integers(0, W + 1, size=B).astype(np.int32)):
        ref = orc.reorder(pats, P, window_len=window_len)
        c = w.make_config(batch=B, window=W)
        step = w.DecodeStep(c)
        wl = None if window_len is None else torch.tensor(window_len, device="cuda")
        step.reorder(torch.tensor(pats, device="cuda"), torch.tensor(toks, device="cuda"), torch.tensor(P, device="cuda"), wl)
        torch.cuda.synchronize()
        for name in ("perm", "inv_perm", "pos_ids", "n_filled", "n_commit"):
            np.testing.assert_array_equal(getattr(step, name).cpu().numpy(), ref[name], err_msg=name)
        np.testing.assert_array_equal(step.tokens_phys.cpu().numpy(), np.take_along_axis(toks, ref["perm"], axis=1))


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("planned,actual", [(100, 600), (2000, 5000), (2000, 2001)])
def test_prefix_beyond_the_planned_bound_is_flagged_and_writes_nothing_out_of_bounds(impl, planned, actual):
    """prefix_len lives on the device and may run ahead of the host's max_prefix_len.  The key split and the
    workspace were sized from the host bound, so the kernels clamp the device value to it, set
    WEDLM_STATUS_BAD_LENGTH and stay inside the workspace: guard bytes behind it keep their pattern, the
    output stays finite, and a second sequence that respects the bound is still computed correctly."""
    import paper_2512_22737_b200 as w
    import parity_util as pu
    cfg = _small_qwen(batch=2, window=8, prefix_lo=planned, prefix_hi=planned, vocab=1000, name="overrun")
    inp = make_step(cfg, seed=planned + actual)
    ref = pu.oracle_step(cfg, inp)
    d = pu.device_inputs(inp)
    # the table of sequence 0 also covers the larger prefix: the extra entries all name a spare page that no
    # sequence owns, so the rows staged at the overrun position land there and disturb nothing
    n_pages_needed = (actual + cfg.window + 15) // 16
    pool = inp["k_cache"].shape[0]
    owned = set(inp["block_table"][inp["block_table"] >= 0].tolist())
    spare = next(pg for pg in range(pool) if pg not in owned)
    n_have = inp["block_table"].shape[1]
    table = torch.zeros(2, max(n_pages_needed, n_have), dtype=torch.int32, device="cuda")
    table[:, :n_have] = d["block_table"].clamp(min=0)
    table[0, n_have:] = spare
    c = w.config_for(cfg, max_pages_per_seq=table.shape[1], num_pages=pool, max_prefix_len=planned, attn_impl=impl)
    step = w.DecodeStep(c)
    need = w.wedlm_window_attn_workspace_bytes(c)
    guard = 1 << 16
    ws_full = torch.full((need + guard,), 0xAB, dtype=torch.uint8, device="cuda")
    prefix = d["prefix_len"].clone()
    prefix[0] = actual
    step.reorder(d["filled"], d["window_tokens"], d["prefix_len"])          # position ids of the planned prefix
    w.wedlm_window_attn(c, d["q"], d["k"], d["v"], d["k_cache"], d["v_cache"], table, prefix, step.pos_ids, step.out,
                        step.kv_slot_idx, ws_full[:need], step.status)
    torch.cuda.synchronize()
    assert int(step.status.item()) & w.binding.WEDLM_STATUS_BAD_LENGTH
    assert not int(step.status.item()) & w.binding.WEDLM_STATUS_WAIT_EXPIRED
    assert bool((ws_full[need:] == 0xAB).all()), "bytes behind the workspace were overwritten"
    got = pu.bf16_from_device(step.out)
    assert np.isfinite(got).all()
    assert pu.attn_vector_error(got[1], ref["out"][1]).max() <= pu.ATTN_REL_TOL


def test_step_is_capturable_in_a_cuda_graph_and_replays_identically():
    """The three calls use only the caller's stream and device-resident sizes: a captured step replayed
    on restored inputs reproduces the eager results bit for bit."""
    import paper_2512_22737_b200 as w
    import parity_util as pu
    cfg = _small_qwen(batch=3, window=16, prefix_lo=100, prefix_hi=900, vocab=8192, boost=14.0, name="graph")
    inp = make_step(cfg, seed=123)
    d = pu.device_inputs(inp)
    c = w.config_for(cfg, max_pages_per_seq=inp["block_table"].shape[1], num_pages=inp["k_cache"].shape[0],
                     max_prefix_len=int(inp["prefix_len"].max()))
    step = w.DecodeStep(c)
    state0 = {k: d[k].clone() for k in ("filled", "window_tokens", "prefix_len")}
    step.run(d)
    torch.cuda.synchronize()
    eager = {k: getattr(step, k).clone() for k in ("out", "argmax", "entropy", "committed_count", "committed_tokens")}
    eager_state = {k: d[k].clone() for k in state0}
    for k, v in state0.items():
        d[k].copy_(v)
    graph = step.capture_graph(d)          # runs once eagerly, then captures once
    for _ in range(2):
        for k, v in state0.items():
            d[k].copy_(v)
        graph.replay()
        torch.cuda.synchronize()
        for k, v in eager.items():
            assert torch.equal(getattr(step, k).view(torch.uint8), v.view(torch.uint8)), k
        for k, v in eager_state.items():
            assert torch.equal(d[k], v), k


def test_a_wait_that_nothing_satisfies_expires_and_reports_status():
    """Failure detection without a fault: the wait gives up after its poll limit, the status word
    carries WEDLM_STATUS_WAIT_EXPIRED, and the context keeps working."""
    import paper_2512_22737_b200 as w
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    w.wedlm_selftest_wait_expiry(20000, status)
    torch.cuda.synchronize()
    assert int(status.item()) == w.binding.WEDLM_STATUS_WAIT_EXPIRED
    # the context is intact: a normal step still runs and matches the oracle
    import parity_util as pu
    cfg = _small_qwen(batch=1, window=8, prefix_lo=40, prefix_hi=40, vocab=1024, name="afterwait")
    pu.full_parity(cfg, make_step(cfg, seed=2))


@pytest.mark.parametrize("impl", IMPLS)
def test_block_wise_commit_mode(impl):
    """WEDLM_COMMIT_BLOCK: nothing is committed unless every active slot is filled."""
    import parity_util as pu
    cfg = _small_qwen(batch=4, window=8, prefix_lo=30, prefix_hi=200, vocab=2048, boost=14.0, boost_prob=0.8,
                      name="blockmode")
    f = np.array([[1, 1, 1, 1, 1, 1, 1, 1], [1, 1, 0, 1, 0, 0, 1, 1], [0, 0, 0, 0, 0, 0, 0, 0], [1, 1, 1, 1, 1, 0, 0, 0]], np.uint8)
    inp = make_step(cfg, seed=51, filled=f)
    r = pu.full_parity(cfg, inp, attn_impl=impl, window_len=[8, 8, 8, 5], remaining_budget=[50, 50, 50, 2],
                       commit_mode="block")
    assert r["step"].committed_count.cpu().tolist() == [8, 0, 0, 5]
