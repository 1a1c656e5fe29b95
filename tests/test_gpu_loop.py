"""Multi-step parity: Streaming Parallel Decoding run through the library on the GPU against the
cache-free fp64 oracle model.  These are the tests that exercise the in-place commit across steps:
rows staged behind the prefix in one step are read back as cache in the next."""
import numpy as np
import pytest
import torch

from oracle import model_oracle as mo
from oracle import wedlm_oracle as orc
from workloads import StepConfig
from workloads.model import TINY, ModelConfig, make_model, make_prompts_and_targets

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("W,tilt,tau", [(1, 0.0, 0.3), (2, 8.0, 0.3), (4, 8.0, 0.5), (8, 30.0, 0.35), (8, 4.0, 2.0), (16, 30.0, 0.35), (5, 14.0, 0.6)])
def test_tiny_model_text_is_token_exact(W, tilt, tau):
    """fp32 kernels vs the fp64 oracle: the committed text, the step count and p_cache agree.
    (tau is kept off the multiples of lambda: with near-zero entropies H + lambda*d lands exactly on a
    threshold such as 0.3 = 3 * 0.1, which is a tie inside the 1e-3 band, not a parity case.)"""
    from paper_2512_22737_b200.loop import StreamingDecoder
    B, P, N = 3, 21, 26
    wts = make_model(TINY)
    pt = make_prompts_and_targets(TINY, B, P, N)
    dec = StreamingDecoder(TINY, wts, batch=B, window=W, max_total_len=P + N, tau=tau, lam=0.1, tilt=tilt,
                           target=pt["target"])
    dec.prefill(pt["prompt"])
    got = dec.generate(N)
    assert int(dec.step_bufs.status.item()) == 0
    steps_ref, n_fwd_ref = 0, 0
    for b in range(B):
        ref = mo.decode(wts, TINY, pt["prompt"][b], pt["target"][b], tilt=tilt, window=W, max_new_tokens=N,
                        conf_mode="entropy", tau=tau, lam=0.1, maxprob_thr=0.9)
        assert got["y"][b] == ref["y"], (b, got["y"][b], ref["y"])
        assert len(ref["y"]) == N
        steps_ref = max(steps_ref, ref["steps"])
        n_fwd_ref += ref["n_fwd"]
    assert got["steps"] == steps_ref
    assert got["n_fwd"] == n_fwd_ref
    assert 0.0 < got["p_cache"] <= 1.0
    if tilt >= 30.0:
        # a strong tilt makes the text the target sequence and several tokens commit per step
        for b in range(B):
            assert got["y"][b] == pt["target"][b, P:P + N].tolist()
        assert got["steps"] < N


def test_tiny_model_step_wise_scheme_w6_is_token_exact():
    """The evaluation setting of Section 6.1: W = 6, lambda = 0.1, one token per step at the lowest adjusted entropy."""
    from paper_2512_22737_b200.loop import StreamingDecoder
    B, P, N, W = 2, 21, 20, 6
    wts = make_model(TINY)
    pt = make_prompts_and_targets(TINY, B, P, N)
    dec = StreamingDecoder(TINY, wts, batch=B, window=W, max_total_len=P + N, tau=float("-inf"), lam=0.1, tilt=5.0,
                           target=pt["target"])
    dec.prefill(pt["prompt"])
    got = dec.generate(N)
    for b in range(B):
        ref = mo.decode(wts, TINY, pt["prompt"][b], pt["target"][b], tilt=5.0, window=W, max_new_tokens=N,
                        conf_mode="entropy", tau=float("-inf"), lam=0.1, maxprob_thr=0.9)
        assert got["y"][b] == ref["y"]
        assert all(t["filled"] <= 1 for t in ref["trace"])
    assert max(got["commits_per_step"]) <= B * W


@pytest.mark.parametrize("W,tilt,tau,T", [(4, 6.0, 0.5, 0.7), (8, 4.0, 2.0, 1.0), (8, 8.0, 0.35, 0.1), (1, 2.0, 0.3, 1.5)])
def test_tiny_model_sampled_text_is_token_exact(W, tilt, tau, T):
    """Sample() at a temperature: the GPU loop and the oracle draw from the same counter-based generator, keyed
    by (seed, sequence, position), so the sampled text agrees token by token as well."""
    from paper_2512_22737_b200.loop import StreamingDecoder
    B, P, N = 3, 21, 26
    seed = (3 << 32) | 77
    wts = make_model(TINY)
    pt = make_prompts_and_targets(TINY, B, P, N)
    dec = StreamingDecoder(TINY, wts, batch=B, window=W, max_total_len=P + N, tau=tau, lam=0.1, tilt=tilt,
                           target=pt["target"], temperature=T, sample_seed=seed)
    dec.prefill(pt["prompt"])
    got = dec.generate(N)
    greedy_same = 0
    for b in range(B):
        ref = mo.decode(wts, TINY, pt["prompt"][b], pt["target"][b], tilt=tilt, window=W, max_new_tokens=N,
                        conf_mode="entropy", tau=tau, lam=0.1, maxprob_thr=0.9, temperature=T,
                        sample_seed=(seed & 0xFFFFFFFF, seed >> 32), seq_index=b)
        assert got["y"][b] == ref["y"], (b, got["y"][b], ref["y"])
        greedy = mo.decode(wts, TINY, pt["prompt"][b], pt["target"][b], tilt=tilt, window=W, max_new_tokens=N,
                           conf_mode="entropy", tau=tau, lam=0.1, maxprob_thr=0.9)
        greedy_same += int(greedy["y"] == ref["y"])
    if T >= 0.7:
        assert greedy_same < B          # the sampled text is not the greedy text


@pytest.mark.parametrize("W,tilt,tau,T", [(8, 8.0, 0.35, 0.0), (4, 6.0, 0.5, 0.7), (1, 0.0, 0.3, 0.0)])
def test_generation_replayed_from_a_cuda_graph_equals_the_eager_loop(W, tilt, tau, T):
    """The whole step (layers, LM head, confidence / commit / refill) captured once and replayed: same text,
    step count and p_cache as the eager loop."""
    from paper_2512_22737_b200.loop import StreamingDecoder
    B, P, N = 3, 21, 26
    wts = make_model(TINY)
    pt = make_prompts_and_targets(TINY, B, P, N)
    outs = []
    for use_graph in (False, True):
        dec = StreamingDecoder(TINY, wts, batch=B, window=W, max_total_len=P + N, tau=tau, lam=0.1, tilt=tilt,
                               target=pt["target"], temperature=T, sample_seed=99)
        dec.prefill(pt["prompt"])
        outs.append(dec.generate(N, use_graph=use_graph))
        assert int(dec.step_bufs.status.item()) == 0
    a, b = outs
    assert a["y"] == b["y"]
    assert a["steps"] == b["steps"] and a["n_fwd"] == b["n_fwd"] and a["commits_per_step"] == b["commits_per_step"]
    assert all(len(y) == N for y in b["y"])


@pytest.mark.parametrize("W,tilt,tau", [(4, 8.0, 0.5), (8, 30.0, 0.35)])
def test_tiny_model_block_wise_baseline_is_token_exact(W, tilt, tau):
    from paper_2512_22737_b200.loop import StreamingDecoder
    B, P, N = 2, 21, 26
    wts = make_model(TINY)
    pt = make_prompts_and_targets(TINY, B, P, N)
    dec = StreamingDecoder(TINY, wts, batch=B, window=W, max_total_len=P + N, tau=tau, lam=0.1, tilt=tilt,
                           target=pt["target"], commit_mode="block")
    dec.prefill(pt["prompt"])
    # prefill windows are fully filled, so the block rule commits them whole as well
    assert dec.prefix_len.cpu().tolist() == [P] * B
    got = dec.generate(N)
    n_fwd_ref = 0
    for b in range(B):
        ref = mo.decode(wts, TINY, pt["prompt"][b], pt["target"][b], tilt=tilt, window=W, max_new_tokens=N,
                        conf_mode="entropy", tau=tau, lam=0.1, maxprob_thr=0.9, block_commit=True)
        assert got["y"][b] == ref["y"]
        n_fwd_ref += ref["n_fwd"]
    assert got["n_fwd"] == n_fwd_ref


def _bits(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16) if t.dtype == torch.bfloat16 else t.cpu().numpy()


@pytest.mark.parametrize("impl", ["tensor", "generic"])
def test_bf16_loop_replays_every_step_against_the_oracle(impl):
    """Qwen-shaped heads (D = 128, G = 4) in bf16: the trajectory is the GPU's own; each step's hot-path
    inputs are captured and the step is recomputed by the oracle (attention of one layer, confidence,
    commit / refill)."""
    import parity_util as pu
    from paper_2512_22737_b200.loop import StreamingDecoder
    m = ModelConfig(name="small_bf16", vocab=4096, hidden=256, n_layers=2, n_q_heads=8, n_kv_heads=2, head_dim=128,
                    ffn=512, dtype="bf16", rope_theta=1.0e6, init_std=0.05)
    B, W, P, N = 4, 16, 70, 48
    wts = make_model(m, seed=5)
    pt = make_prompts_and_targets(m, B, P, N, seed=5)
    dec = StreamingDecoder(m, wts, batch=B, window=W, max_total_len=P + N, tau=0.3, lam=0.1, tilt=14.0,
                           target=pt["target"], attn_impl=impl)
    dec.prefill(pt["prompt"])
    assert dec.prefix_len.cpu().tolist() == [P] * B
    dec.start(N)
    scfg = StepConfig(name="replay", batch=B, window=W, n_q_heads=m.n_q_heads, n_kv_heads=m.n_kv_heads,
                      head_dim=m.head_dim, vocab=m.vocab, dtype="bf16", rope_theta=m.rope_theta, tau=0.3, lam=0.1)
    ys = [[] for _ in range(B)]
    worst, excluded, steps = 0.0, 0, 0
    while int(dec.window_len.sum().item()) > 0 and steps < 200:
        layer = steps % m.n_layers
        cc, ct, cap = dec.step(capture_layer=layer)
        inp = dict(filled=cap["filled"].cpu().numpy(), window_tokens=cap["window_tokens"].cpu().numpy(),
                   prefix_len=cap["prefix_len"].cpu().numpy(), block_table=dec.block_table.cpu().numpy(),
                   k_cache=_bits(cap["k_cache"]), v_cache=_bits(cap["v_cache"]), q=_bits(cap["q"]), k=_bits(cap["k"]),
                   v=_bits(cap["v"]), logits=_bits(cap["logits"]))
        wl, bud = cap["window_len"].cpu().numpy(), cap["budget"].cpu().numpy()
        ref = pu.oracle_step(scfg, inp, window_len=wl, remaining_budget=bud)
        pu.check_reorder(dec.step_bufs, ref)
        err = pu.attn_vector_error(pu.bf16_from_device(cap["out"]), ref["out"])
        # rows of inactive slots (a window that is running out) are not part of the contract
        for b in range(B):
            assert err[b, : wl[b]].max(initial=0.0) <= pu.ATTN_REL_TOL, (steps, b, err[b])
            worst = max(worst, float(err[b, : wl[b]].max(initial=0.0)))
        np.testing.assert_array_equal(cap["kv_slot_idx"].cpu().numpy(), ref["kv_slot_idx"])
        d = dict(window_tokens=dec.window_tokens, filled=dec.filled, prefix_len=dec.prefix_len,
                 window_len=dec.window_len, remaining_budget=dec.budget)
        excluded += pu.check_confidence_and_commit(scfg, dec.step_bufs, d, inp, ref, wl)
        cch, cth = cc.cpu().numpy(), ct.cpu().numpy()
        for b in range(B):
            ys[b].extend(cth[b, : cch[b]].tolist())
        steps += 1
    assert int(dec.step_bufs.status.item()) == 0
    for b in range(B):
        assert len(ys[b]) == N
        assert ys[b] == pt["target"][b, P:P + N].tolist()          # tilt 14 dominates a random-init model
    assert steps < N                                                  # several tokens per step
    print(f"{impl}: {steps} steps for {N} tokens, worst attention error {worst:.2e}, excluded decisions {excluded}")


def test_fused_lm_head_loop_writes_the_same_text():
    """The loop with the LM head fused into the confidence call (no logits tensor) against the loop that
    materialises bf16 logits: same committed text when the tilt decides the tokens, same number of tokens."""
    from paper_2512_22737_b200.loop import StreamingDecoder
    m = ModelConfig(name="small_bf16", vocab=4096, hidden=256, n_layers=2, n_q_heads=8, n_kv_heads=2, head_dim=128,
                    ffn=512, dtype="bf16", rope_theta=1.0e6, init_std=0.05)
    B, W, P, N = 3, 16, 40, 40
    wts = make_model(m, seed=7)
    pt = make_prompts_and_targets(m, B, P, N, seed=7)
    outs = []
    for fused in (False, True):
        dec = StreamingDecoder(m, wts, batch=B, window=W, max_total_len=P + N, tau=0.35, lam=0.1, tilt=16.0,
                               target=pt["target"], fused_lm_head=fused)
        dec.prefill(pt["prompt"])
        outs.append(dec.generate(N))
    for b in range(B):
        assert outs[1]["y"][b] == pt["target"][b, P:P + N].tolist()
        assert outs[0]["y"][b] == outs[1]["y"][b]
    assert outs[1]["steps"] < N
    # fp32 logits against bf16-rounded ones can flip a borderline selection, not change the pace of decoding
    assert abs(outs[0]["steps"] - outs[1]["steps"]) <= 2
