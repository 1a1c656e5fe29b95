"""The workspace-free confidence/commit call against the regular one.

`wedlm_confidence_commit_static` serves hosts that cannot allocate device memory while running (all
of HBM already belongs to a cache pool, or allocator calls are banned after warm-up): its scratch is
a fixed array inside the library.  Here it is called through the C ABI twice in a row, on two
different window states, and every output is compared with what `wedlm_confidence_commit` produces
from the same inputs with a caller-provided workspace.  The second call runs on top of whatever the
first one left in the shared array, which must not matter.

This file sorts last so that a run that stops at the first failure has already run everything else.
"""
import numpy as np
import pytest
import torch

from workloads import get_config, make_step

pytestmark = pytest.mark.gpu


def _run_both(cfg, inp, temperature=0.0, check_oracle=False, check_no_alloc=False):
    import paper_2512_22737_b200 as w
    import parity_util as pu
    c = w.config_for(cfg, max_pages_per_seq=inp["block_table"].shape[1], num_pages=inp["k_cache"].shape[0],
                     max_prefix_len=int(inp["prefix_len"].max()), sample_temperature=temperature, sample_seed=1234567)
    results = []
    for variant in ("workspace", "static"):
        d = pu.device_inputs(inp)
        step = w.DecodeStep(c)
        step.reorder(d["filled"], d["window_tokens"], d["prefix_len"])
        if variant == "workspace":
            step.confidence_commit(d["logits"], d["window_tokens"], d["filled"], d["prefix_len"])
        else:
            torch.cuda.synchronize()
            free_before, _ = torch.cuda.mem_get_info()
            reserved_before = torch.cuda.memory_reserved()
            w.wedlm_confidence_commit_static(
                c, d["logits"], step.perm, step.n_filled, step.n_commit, d["window_tokens"], d["filled"],
                d["prefix_len"], None, None, step.argmax, step.maxprob, step.entropy, step.lse,
                step.committed_tokens, step.committed_count, step.filled_count)
            torch.cuda.synchronize()
            if check_no_alloc:
                # not the first call on this device (the array is already materialised and its address known):
                # neither the driver's free memory nor torch's pool may have moved
                assert torch.cuda.mem_get_info()[0] == free_before
                assert torch.cuda.memory_reserved() == reserved_before
        torch.cuda.synchronize()
        if check_oracle and temperature == 0.0:
            # the static call against the oracle itself, not only against the other CUDA path
            ref = pu.oracle_step(cfg, inp, with_attention=False)
            pu.check_reorder(step, ref)
            pu.check_confidence_and_commit(cfg, step, d, inp, ref)
        results.append(dict(
            argmax=step.argmax.cpu().numpy(), maxprob=step.maxprob.cpu().numpy(), entropy=step.entropy.cpu().numpy(),
            lse=step.lse.cpu().numpy(), committed_tokens=step.committed_tokens.cpu().numpy(),
            committed_count=step.committed_count.cpu().numpy(), filled_count=step.filled_count.cpu().numpy(),
            window_tokens=d["window_tokens"].cpu().numpy(), filled=d["filled"].cpu().numpy(),
            prefix_len=d["prefix_len"].cpu().numpy()))
    return results


def _compare(a, b):
    import parity_util as pu
    for k in ("argmax", "committed_tokens", "committed_count", "filled_count", "window_tokens", "filled", "prefix_len"):
        np.testing.assert_array_equal(a[k], b[k], err_msg=k)
    for k in ("maxprob", "entropy", "lse"):
        x, y = a[k].astype(np.float64), b[k].astype(np.float64)
        assert (np.isnan(x) == np.isnan(y)).all(), k
        ok = ~np.isnan(x)
        assert (np.abs(x[ok] - y[ok]) <= pu.CONF_REL_TOL * np.maximum(np.abs(x[ok]), 1e-3)).all(), k


def test_static_scratch_variant_matches_the_workspace_variant_on_two_calls_in_a_row():
    base = get_config("cfg2_qwen_b1")
    first = base.replace(batch=3, window=16, prefix_lo=20, prefix_hi=90, boost=16.4, boost_prob=0.7, name="noalloc1")
    second = base.replace(batch=5, window=8, vocab=50000, prefix_lo=5, prefix_hi=40, boost=20.4, boost_prob=0.5,
                          obs_prob_lo=0.6, obs_prob_hi=0.6, name="noalloc2")
    for n, (cfg, seed) in enumerate(((first, 71), (second, 72))):
        inp = make_step(cfg, seed=seed)
        with_ws, static = _run_both(cfg, inp, check_oracle=True, check_no_alloc=(n > 0))
        assert (static["argmax"] >= 0).any()
        _compare(with_ws, static)


def test_static_scratch_variant_with_a_sampling_temperature_twice_in_a_row():
    """With a temperature the shared array also holds the sampling pass's lists and counters (selected rows,
    per-row best score, chunk counts).  Two calls back to back, the second on top of the first one's
    leftovers: each must draw exactly the tokens the workspace variant draws from the same seed."""
    base = get_config("cfg2_qwen_b1")
    first = base.replace(batch=4, window=16, vocab=30000, prefix_lo=20, prefix_hi=90, boost=16.4, boost_prob=0.7,
                         name="noalloc_t1")
    second = base.replace(batch=2, window=8, vocab=50000, prefix_lo=5, prefix_hi=40, boost=14.0, boost_prob=0.5,
                          obs_prob_lo=0.2, obs_prob_hi=0.2, name="noalloc_t2")
    for cfg, seed, temp in ((first, 81, 0.7), (second, 82, 1.5)):
        inp = make_step(cfg, seed=seed)
        with_ws, static = _run_both(cfg, inp, temperature=temp)
        assert (static["filled_count"] > 0).any()
        _compare(with_ws, static)


def test_sizes_beyond_the_built_in_array_are_refused():
    import paper_2512_22737_b200 as w
    # 64 * 1024 rows * 19 chunks * 16 B is far beyond 4 MiB
    c = w.make_config(batch=64, window=1024, vocab=151936, dtype="bf16")
    assert w.wedlm_confidence_workspace_bytes(c) > w.binding.WEDLM_STATIC_SCRATCH_BYTES
    e = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(w.WedlmError) as err:
        w.wedlm_confidence_commit_static(c, torch.zeros(8, dtype=torch.bfloat16, device="cuda"), e, e, e, e,
                                         torch.zeros(1, dtype=torch.uint8, device="cuda"), e, None, None,
                                         None, None, None, None, None, None, None)
    assert err.value.code == w.binding.WEDLM_ERR_STATIC_SCRATCH
    assert "scratch" in str(err.value)
