"""The seeded generators: determinism, shapes, and the distributions the configs state."""
import numpy as np
import torch

from workloads import CONFIGS, bf16_bits, bf16_to_f32, get_config, make_step


def test_bf16_round_trip_matches_torch():
    x = np.random.default_rng(0).standard_normal(10000).astype(np.float32) * 37.0
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    np.testing.assert_array_equal(bf16_to_f32(bf16_bits(x)), ref)


def test_same_seed_same_arrays_and_other_seed_differs():
    cfg = get_config("cfg1_tiny")
    a, b, c = make_step(cfg), make_step(cfg), make_step(cfg, seed=7)
    for k in a:
        np.testing.assert_array_equal(a[k], b[k])
    assert not np.array_equal(a["logits"], c["logits"])


def test_cfg2_shapes_and_page_table():
    cfg = get_config("cfg2_qwen_b1")
    s = make_step(cfg)
    B, W = cfg.batch, cfg.window
    assert s["q"].shape == (B, W, 32, 128) and s["q"].dtype == np.uint16
    assert s["k"].shape == (B, W, 8, 128) and s["logits"].shape == (B, W, 151936)
    assert s["prefix_len"].tolist() == [2048]
    n_pages = (2048 + W + 15) // 16
    used = s["block_table"][0, :n_pages]
    assert (used >= 0).all() and len(set(used.tolist())) == n_pages and used.max() < s["k_cache"].shape[0]
    # mask slots hold the mask id, filled slots a regular token
    tok, f = s["window_tokens"], s["filled"]
    assert (tok[f == 0] == cfg.mask_token_id).all() and (tok[f == 1] < cfg.mask_token_id).all()
    # boosted rows: the target's logit stands out by about the boost
    x = bf16_to_f32(s["logits"])
    t = s["targets"]
    rows = np.nonzero(t[0] >= 0)[0]
    assert 2 <= len(rows) <= 14
    assert all(x[0, r, t[0, r]] > 4.0 for r in rows)
    assert abs(float(x.std()) - 1.0) < 0.01


def test_clustered_runs_pattern_statistics():
    cfg = get_config("cfg4_long").replace(batch=2000, prefix_lo=0, prefix_hi=0, vocab=8, n_q_heads=1,
                                          n_kv_heads=1, head_dim=2)
    s = make_step(cfg, with_logits=False)
    f = s["filled"]
    assert abs(f.mean() - 0.5) < 0.02
    # mean run length of interior runs is near 4
    runs = []
    for row in f:
        edges = np.nonzero(np.diff(row))[0]
        runs += np.diff(edges).tolist()
    assert 3.5 < np.mean(runs) < 4.5


def test_all_named_configs_exist():
    assert set(CONFIGS) == {"cfg1_tiny", "cfg2_qwen_b1", "cfg3_batched", "cfg4_long"}
