"""wedlm_step_host: the whole step driven from host buffers, against the oracle.

The device workspace is poisoned before the call (0xFF bytes are NaN in bf16 and fp32), so a logits row
that the step reads but the call failed to send would surface as NaN statistics."""
import numpy as np
import pytest
import torch

import paper_2512_22737_b200 as w
import parity_util as pu
from workloads import get_config, make_step

pytestmark = pytest.mark.gpu


def _host(a):
    t = torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else np.ascontiguousarray(a)).clone()
    return t.pin_memory()


def _run(cfg, inp, window_len=None, budget=None, attn_impl="auto"):
    c = w.config_for(cfg, max_pages_per_seq=inp["block_table"].shape[1], num_pages=inp["k_cache"].shape[0],
                     max_prefix_len=int(inp["prefix_len"].max()), batch=inp["filled"].shape[0], attn_impl=attn_impl)
    B, W = inp["filled"].shape
    h = {k: _host(inp[k]) for k in ("filled", "window_tokens", "prefix_len", "block_table", "q", "k", "v", "logits")}
    h_wl = None if window_len is None else _host(np.asarray(window_len, np.int32))
    h_rb = None if budget is None else _host(np.asarray(budget, np.int32))
    ct = torch.full((B, W), -9, dtype=torch.int32).pin_memory()
    cc = torch.full((B,), -9, dtype=torch.int32).pin_memory()
    fc = torch.full((B,), -9, dtype=torch.int32).pin_memory()
    kc, vc = w.to_device(inp["k_cache"]), w.to_device(inp["v_cache"])
    ws = torch.full((w.wedlm_step_host_workspace_bytes(c),), 0xFF, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out_ptr = w.wedlm_step_host(c, h["filled"], h["window_tokens"], h["prefix_len"], h_wl, h_rb, h["block_table"], h["q"],
                                h["k"], h["v"], h["logits"], kc, vc, ct, cc, fc, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    # attention output: a view into the workspace at the returned address
    off = out_ptr - ws.data_ptr()
    n_out = B * W * cfg.n_q_heads * cfg.head_dim
    elem = 2 if cfg.dtype == "bf16" else 4
    raw = ws[off: off + n_out * elem]
    out = raw.view(torch.bfloat16 if cfg.dtype == "bf16" else torch.float32).view(B, W, cfg.n_q_heads, cfg.head_dim)
    return dict(h=h, wl=h_wl, rb=h_rb, ct=ct, cc=cc, fc=fc, out=out.to(torch.float64).cpu().numpy(), kc=kc, vc=vc)


def _check(cfg, inp, r, window_len=None, budget=None):
    ref = pu.oracle_step(cfg, inp, window_len=window_len, remaining_budget=budget)
    B, W = inp["filled"].shape
    err = pu.attn_vector_error(r["out"], ref["out"])
    for b in range(B):
        L = W if window_len is None else int(window_len[b])
        assert err[b, :L].max(initial=0.0) <= pu.ATTN_REL_TOL
    excluded = 0
    for b in range(B):
        ps = ref["per_seq"][b]
        n = ps["committed_count"]
        assert int(r["cc"][b]) == n
        assert r["ct"][b, :n].tolist() == ps["committed_tokens"]
        assert int(r["h"]["prefix_len"][b]) == ps["prefix_len"]
        if window_len is not None:
            assert int(r["wl"][b]) == ps["window_len"]
        if budget is not None:
            assert int(r["rb"][b]) == ps["remaining_budget"]
        sc = np.asarray(ps["scores"], dtype=np.float64)
        thr = cfg.tau if cfg.conf_mode == "entropy" else -cfg.maxprob_thr
        tie = bool(len(sc) and (np.abs(sc - thr) <= pu.TIE_BAND * max(1.0, abs(thr))).any())
        if len(sc) > 1 and not (sc <= thr).any():
            srt = np.sort(sc)
            tie = tie or bool(srt[1] - srt[0] <= pu.TIE_BAND * max(1.0, abs(srt[0])))
        if tie:
            excluded += 1
            continue
        assert int(r["fc"][b]) == ps["filled_count"]
        assert r["h"]["window_tokens"][b].tolist() == ps["window_tokens"]
        assert r["h"]["filled"][b].tolist() == ps["filled"]
    return excluded


def test_tiny_fp32_from_host_buffers():
    cfg = get_config("cfg1_tiny").replace(conf_mode="entropy", tau=7.5, batch=3)
    inp = make_step(cfg, seed=5)
    assert _check(cfg, inp, _run(cfg, inp)) <= 1


@pytest.mark.parametrize("impl", ["tensor", "generic"])
def test_bf16_batches_with_boosts(impl):
    cfg = get_config("cfg2_qwen_b1").replace(vocab=20000, batch=5, window=16, prefix_lo=10, prefix_hi=600, boost=14.0,
                                            boost_prob=0.6, name="host")
    inp = make_step(cfg, seed=9)
    assert _check(cfg, inp, _run(cfg, inp, attn_impl=impl)) <= 1


def test_short_windows_and_budgets_only_send_the_rows_in_use():
    cfg = get_config("cfg2_qwen_b1").replace(vocab=10007, batch=4, window=8, prefix_lo=30, prefix_hi=90, tau=50.0, name="hostwl")
    inp = make_step(cfg, seed=21)
    wl = np.array([8, 5, 1, 0], np.int32)
    rb = np.array([3, 0, 9, 2], np.int32)
    _check(cfg, inp, _run(cfg, inp, window_len=wl, budget=rb), window_len=wl, budget=rb)


def test_matches_the_device_path_bit_for_bit():
    cfg = get_config("cfg2_qwen_b1").replace(vocab=32000, batch=6, prefix_lo=100, prefix_hi=900, boost=15.0, boost_prob=0.5,
                                            name="hostdev")
    inp = make_step(cfg, seed=33)
    r = _run(cfg, inp)
    step, d = pu.run_gpu_step(cfg, inp)
    assert torch.equal(r["h"]["window_tokens"], d["window_tokens"].cpu())
    assert torch.equal(r["h"]["filled"], d["filled"].cpu())
    assert torch.equal(r["cc"], step.committed_count.cpu())
    np.testing.assert_array_equal(r["out"], step.out.to(torch.float64).cpu().numpy())


def test_workspace_too_small_and_bad_config_are_refused_on_the_host():
    cfg = get_config("cfg1_tiny")
    inp = make_step(cfg, seed=1)
    c = w.config_for(cfg, max_pages_per_seq=inp["block_table"].shape[1], num_pages=inp["k_cache"].shape[0],
                     max_prefix_len=int(inp["prefix_len"].max()))
    need = w.wedlm_step_host_workspace_bytes(c)
    assert need > 0
    h = {k: _host(inp[k]) for k in ("filled", "window_tokens", "prefix_len", "block_table", "q", "k", "v", "logits")}
    kc, vc = w.to_device(inp["k_cache"]), w.to_device(inp["v_cache"])
    out = torch.zeros(8, dtype=torch.int32).pin_memory()
    small = torch.empty(need - 256, dtype=torch.uint8, device="cuda")
    with pytest.raises(w.WedlmError) as ei:
        w.wedlm_step_host(c, h["filled"], h["window_tokens"], h["prefix_len"], None, None, h["block_table"], h["q"], h["k"],
                          h["v"], h["logits"], kc, vc, out, out[:1], None, small)
    assert ei.value.code == -3


def test_step_from_host_hidden_states_with_the_lm_head_on_the_device():
    """wedlm_step_host_lmhead: hidden states come from the host, the output embedding is resident; the oracle gets
    logits = hidden . lm_head^T in float64 from the same bf16 bit patterns."""
    from oracle import wedlm_oracle as orc
    from workloads import bf16_bits
    cfg = get_config("cfg2_qwen_b1").replace(batch=3, window=16, vocab=6000, prefix_lo=40, prefix_hi=300, tau=0.3, name="host_lmhead")
    inp = make_step(cfg, seed=91, with_logits=False)
    B, W, V, H = 3, 16, cfg.vocab, 256
    g = np.random.default_rng(91)
    hid = bf16_bits(g.standard_normal((B, W, H)).astype(np.float32).reshape(-1)).reshape(B, W, H)
    emb = bf16_bits((g.standard_normal((V, H)) * (2.0 / np.sqrt(H))).astype(np.float32).reshape(-1)).reshape(V, H)
    tilt_ids = g.integers(0, V - 1, size=(B, W)).astype(np.int32)
    tilt_ids[g.random((B, W)) < 0.3] = -1
    boost = 12.0
    logits = orc.to_f64(hid) @ orc.to_f64(emb).T
    bb, ww = np.nonzero(tilt_ids >= 0)
    logits[bb, ww, tilt_ids[bb, ww]] += boost
    inp["logits"] = logits
    c = w.config_for(cfg, max_pages_per_seq=inp["block_table"].shape[1], num_pages=inp["k_cache"].shape[0],
                     max_prefix_len=int(inp["prefix_len"].max()), batch=B)
    h = {k: _host(inp[k]) for k in ("filled", "window_tokens", "prefix_len", "block_table", "q", "k", "v")}
    h_hid, h_tilt = _host(hid), _host(tilt_ids)
    ct = torch.full((B, W), -9, dtype=torch.int32).pin_memory()
    cc = torch.full((B,), -9, dtype=torch.int32).pin_memory()
    fc = torch.full((B,), -9, dtype=torch.int32).pin_memory()
    kc, vc = w.to_device(inp["k_cache"]), w.to_device(inp["v_cache"])
    ws = torch.full((w.wedlm_step_host_lmhead_workspace_bytes(c, H),), 0xFF, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out_ptr = w.wedlm_step_host_lmhead(c, h["filled"], h["window_tokens"], h["prefix_len"], None, None, h["block_table"],
                                       h["q"], h["k"], h["v"], h_hid, w.to_device(emb), h_tilt, boost, kc, vc, ct, cc, fc, ws,
                                       status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    off = out_ptr - ws.data_ptr()
    out = ws[off: off + B * W * cfg.n_q_heads * cfg.head_dim * 2].view(torch.bfloat16).view(B, W, cfg.n_q_heads, cfg.head_dim)
    r = dict(h=h, wl=None, rb=None, ct=ct, cc=cc, fc=fc, out=out.to(torch.float64).cpu().numpy())
    _check(cfg, inp, r)
    # the call refuses a hidden size the tensor-core tiles cannot cover
    assert w.wedlm_step_host_lmhead_workspace_bytes(c, 100) == 0
