"""Helpers of the GPU parity tests: run one step through the C-ABI binding, run the oracle on the
same arrays, compare item by item under the stated tolerances."""
from __future__ import annotations

from typing import Dict, Optional

import numpy as np
import torch

import paper_2512_22737_b200 as w
from oracle import wedlm_oracle as orc

# Tolerances of the parity comparison:
ATTN_REL_TOL = 1e-2      # per output vector: max|gpu - ref| / max|ref|, bf16 in / fp32 accumulate
CONF_REL_TOL = 1e-3      # entropy, lse, max-prob; entropy/lse with an absolute floor of 1e-3 * 1e-3
TIE_BAND = 1e-3          # decisions whose fp64 margin is inside this band are excluded and counted


def device_inputs(inp: Dict[str, np.ndarray]) -> Dict[str, torch.Tensor]:
    return {k: w.to_device(v) for k, v in inp.items() if k != "targets"}


def bf16_from_device(t: torch.Tensor) -> np.ndarray:
    """CUDA tensor -> float64 numpy (exact widening)."""
    return t.detach().to(torch.float64).cpu().numpy()


def run_gpu_step(cfg, inp, *, attn_impl="auto", window_len=None, remaining_budget=None, commit_mode="streaming"):
    """One full step on the GPU.  Returns (DecodeStep with outputs, device dict with the updated
    window state and cache)."""
    d = device_inputs(inp)
    c = w.config_for(cfg, max_pages_per_seq=inp["block_table"].shape[1], num_pages=inp["k_cache"].shape[0],
                     max_prefix_len=int(inp["prefix_len"].max()) if len(inp["prefix_len"]) else 0,
                     attn_impl=attn_impl, batch=inp["filled"].shape[0], commit_mode=commit_mode)
    step = w.DecodeStep(c)
    wl = None if window_len is None else torch.tensor(window_len, dtype=torch.int32, device="cuda")
    rb = None if remaining_budget is None else torch.tensor(remaining_budget, dtype=torch.int32, device="cuda")
    step.run(d, wl, rb)
    torch.cuda.synchronize()
    d["window_len"] = wl
    d["remaining_budget"] = rb
    return step, d


def oracle_step(cfg, inp, *, window_len=None, remaining_budget=None, with_attention=True, block_commit=False):
    return orc.step(inp, theta=cfg.rope_theta, conf_mode=cfg.conf_mode, tau=cfg.tau, lam=cfg.lam,
                    maxprob_thr=cfg.maxprob_thr, mask_token_id=cfg.mask_token_id, page_size=cfg.page_size,
                    window_len=window_len, remaining_budget=remaining_budget, with_attention=with_attention,
                    block_commit=block_commit)


def attn_vector_error(got: np.ndarray, ref: np.ndarray) -> np.ndarray:
    """Per output vector (last axis): max|got - ref| / max|ref|."""
    num = np.abs(got - ref).max(axis=-1)
    den = np.abs(ref).max(axis=-1)
    return num / np.maximum(den, 1e-30)


def check_reorder(step, ref):
    for name in ("perm", "inv_perm", "pos_ids", "n_filled", "n_commit", "tokens_phys"):
        np.testing.assert_array_equal(getattr(step, name).cpu().numpy(), ref[name], err_msg=name)


def staged_rows(cache: torch.Tensor, slots: np.ndarray, page: int) -> np.ndarray:
    """Cache rows at the given slots (page * page_size + offset), gathered on the device -> float64
    [..., Hkv, D].  Avoids widening a whole gigabyte-sized cache on the host."""
    flat = torch.as_tensor(np.asarray(slots).reshape(-1), dtype=torch.int64, device=cache.device)
    rows = cache[flat // page, :, flat % page]                    # [N, Hkv, D]
    return bf16_from_device(rows).reshape(tuple(np.asarray(slots).shape) + tuple(rows.shape[1:]))


def check_attention(cfg, step, d, inp, ref, rows_active=None):
    """Every output vector within tolerance; slot indices exact; every staged V row bit-exact and every
    staged K row within one bf16 ulp (plus the fp32 rotation noise) of the rounded oracle value."""
    got = bf16_from_device(step.out)
    err = attn_vector_error(got, ref["out"])
    assert np.isfinite(got).all()
    assert err.max() <= ATTN_REL_TOL, f"attention error {err.max():.3e} at {np.unravel_index(err.argmax(), err.shape)}"
    np.testing.assert_array_equal(step.kv_slot_idx.cpu().numpy(), ref["kv_slot_idx"])
    assert int(step.status.item()) == 0
    page = cfg.page_size
    kc = staged_rows(d["k_cache"], ref["kv_slot_idx"], page)      # [B, W, Hkv, D]
    vc = staged_rows(d["v_cache"], ref["kv_slot_idx"], page)
    v_in = orc.to_f64(inp["v"])
    k_in = orc.to_f64(inp["k"])
    np.testing.assert_array_equal(vc, v_in)
    want = ref["k_rot"]
    if cfg.dtype == "bf16":
        # one bf16 ulp of the value, plus the fp32 noise of the rotation itself (a*cos - b*sin
        # can cancel to a result far smaller than a and b): 2^-20 of the row's largest input
        ulp = np.abs(want) * 2.0 ** -7 + np.abs(k_in).max(axis=(2, 3), keepdims=True) * 2.0 ** -20
        assert (np.abs(kc - orc.round_to_bf16(want)) <= ulp).all()
    else:
        np.testing.assert_allclose(kc, want, rtol=2e-6, atol=2e-6)
    return float(err.max())


def check_confidence_and_commit(cfg, step, d, inp, ref, window_len=None, tie_seqs=()):
    """Statistics within tolerance on every active mask row; integer results exact.  Sequences whose
    selection hinges on a margin inside the tie band (and those the caller names in `tie_seqs`, e.g.
    because an arg-max was decided inside the logit band) are excluded from the comparison of this
    step's fills and counted; everything else about them is still compared."""
    B, W = inp["filled"].shape
    am = step.argmax.cpu().numpy()
    ent = step.entropy.cpu().numpy().astype(np.float64)
    mp = step.maxprob.cpu().numpy().astype(np.float64)
    lse = step.lse.cpu().numpy().astype(np.float64)
    np.testing.assert_array_equal(am, ref["argmax"])
    active = ~np.isnan(ref["entropy"])
    assert (np.isnan(ent) == ~active).all()
    if active.any():
        e_ref, m_ref, l_ref = ref["entropy"][active], ref["maxprob"][active], ref["lse"][active]
        assert (np.abs(ent[active] - e_ref) <= CONF_REL_TOL * np.maximum(np.abs(e_ref), 1e-3)).all(), \
            np.abs(ent[active] - e_ref).max()
        assert (np.abs(lse[active] - l_ref) <= CONF_REL_TOL * np.maximum(np.abs(l_ref), 1e-3)).all()
        assert (np.abs(mp[active] - m_ref) <= CONF_REL_TOL * m_ref).all()
    cc = step.committed_count.cpu().numpy()
    ct = step.committed_tokens.cpu().numpy()
    fc = step.filled_count.cpu().numpy()
    tok = d["window_tokens"].cpu().numpy()
    fil = d["filled"].cpu().numpy()
    pl = d["prefix_len"].cpu().numpy()
    wl = None if d.get("window_len") is None else d["window_len"].cpu().numpy()
    rb = None if d.get("remaining_budget") is None else d["remaining_budget"].cpu().numpy()
    excluded = 0
    for b in range(B):
        ps = ref["per_seq"][b]
        n = ps["committed_count"]
        assert cc[b] == n
        assert ct[b, :n].tolist() == ps["committed_tokens"] and (ct[b, n:] == -1).all()
        assert pl[b] == ps["prefix_len"]
        if wl is not None:
            assert wl[b] == ps["window_len"]
        if rb is not None:
            assert rb[b] == ps["remaining_budget"]
        # tie band on the decision
        sc = np.asarray(ps["scores"], dtype=np.float64)
        tie = False
        if len(sc):
            if cfg.conf_mode == "entropy":
                thr, val = cfg.tau, sc
            else:
                thr, val = cfg.maxprob_thr, -sc
            if np.isfinite(thr):
                tie = bool((np.abs(val - thr) <= TIE_BAND * max(1.0, abs(thr))).any())
            passed = (val <= thr) if cfg.conf_mode == "entropy" else (val >= thr)
            if not passed.any() and len(sc) > 1:
                srt = np.sort(sc)
                tie = tie or bool(srt[1] - srt[0] <= TIE_BAND * max(1.0, abs(srt[0])))
        if tie or b in tie_seqs:
            excluded += 1
            continue
        assert fc[b] == ps["filled_count"]
        assert tok[b].tolist() == ps["window_tokens"], (b, tok[b].tolist(), ps["window_tokens"])
        assert fil[b].tolist() == ps["filled"]
    return excluded


def full_parity(cfg, inp, *, attn_impl="auto", window_len=None, remaining_budget=None, commit_mode="streaming"):
    step, d = run_gpu_step(cfg, inp, attn_impl=attn_impl, window_len=window_len, remaining_budget=remaining_budget,
                           commit_mode=commit_mode)
    ref = oracle_step(cfg, inp, window_len=window_len, remaining_budget=remaining_budget,
                      block_commit=(commit_mode == "block"))
    check_reorder(step, ref)
    err = check_attention(cfg, step, d, inp, ref)
    excluded = check_confidence_and_commit(cfg, step, d, inp, ref, window_len)
    return dict(attn_err=err, excluded=excluded, step=step, ref=ref)
